"""Host-side checks that need no GPU: the library builds, exports every declared symbol,
and rejects invalid arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2210_15458_b200 import _build, binding
    _build.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "arith_sampling.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(as_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_2210_15458_b200 import binding
    names = _declared()
    assert "as_step" in names and "as_lattice_codes" in names and "as_decode_bigram" in names
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names
    assert L.as_version() >= 1000


def test_invalid_arguments_are_rejected_on_the_host(L):
    from paper_2210_15458_b200 import binding as B
    one = ctypes.c_double(0.0)
    p = ctypes.addressof(one)
    assert L.as_lattice_codes(0, 0.5, p, None) == B.ERR_INVALID_ARG
    assert b"N" in L.as_last_error()
    assert L.as_lattice_codes(4, 1.0, p, None) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes(4, float("nan"), p, None) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes(4, 0.5, None, None) == B.ERR_INVALID_ARG
    sl = lambda **k: L.as_step_lattice(p, 0, k.get("lanes", 2), 2, 2, k.get("N", 4), k.get("u", 0.5), k.get("j0", 0),
                                       1.0, 0, 1.0, p, p, None, None)
    assert sl(N=0) == B.ERR_INVALID_ARG and sl(u=1.0) == B.ERR_INVALID_ARG and sl(j0=-1) == B.ERR_INVALID_ARG
    assert sl(j0=3) == B.ERR_INVALID_ARG and sl(lanes=5) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes_variant(4, 0.5, 7, p, None) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes_variant(0, 0.5, 1, p, None) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes_variant(4, 1.0, 1, p, None) == B.ERR_INVALID_ARG
    assert L.as_lattice_codes_variant(4, 0.5, 2, None, None) == B.ERR_INVALID_ARG
    step = lambda **k: L.as_step(k.get("logits", p), k.get("dtype", 0), k.get("lanes", 1), k.get("V", 2),
                                 k.get("ld", 2), k.get("codes", p), k.get("temp", 1.0), 0,
                                 k.get("top_p", 1.0), k.get("tokens", p), k.get("out", p), None, None)
    assert step(logits=None) == B.ERR_INVALID_ARG
    assert step(dtype=7) == B.ERR_INVALID_ARG
    assert step(lanes=-1) == B.ERR_INVALID_ARG
    assert step(V=0) == B.ERR_INVALID_ARG
    assert step(V=(1 << 20) + 1, ld=(1 << 20) + 1) == B.ERR_UNSUPPORTED
    assert step(ld=1) == B.ERR_INVALID_ARG
    assert step(temp=0.0) == B.ERR_INVALID_ARG
    assert step(temp=float("inf")) == B.ERR_INVALID_ARG
    assert step(top_p=float("nan")) == B.ERR_INVALID_ARG
    assert step(codes=None) == B.ERR_INVALID_ARG
    assert step(logits=p + 1) == B.ERR_INVALID_ARG
    assert L.as_decode_bigram(p, 0, 2, 2, p, 1, 0, 0.5, 4, 0, 1.0, 0, 1.0, p, p, None, None, None) == B.ERR_INVALID_ARG
    assert L.as_decode_bigram(p, 0, 2, 2, p, 1, 4, 1.5, 4, 0, 1.0, 0, 1.0, p, p, None, None, None) == B.ERR_INVALID_ARG
    assert L.as_decode_bigram(p, 0, 2, 2, p, 1, 4, 0.5, -1, 0, 1.0, 0, 1.0, p, p, None, None, None) == B.ERR_INVALID_ARG
    assert L.as_decode_bigram_codes(p, 0, 2, 2, p, None, 1, 4, 0, 1.0, 0, 1.0, p, p, None, None, None) == B.ERR_INVALID_ARG
    enc = lambda **k: L.as_encode_bigram(k.get("table", p), 0, 2, 2, k.get("prev", p), k.get("seq", p), p,
                                         k.get("lanes", 1), k.get("T", 4), k.get("temp", 1.0), 0, 1.0,
                                         k.get("lo", p), p, None, None)
    assert enc(lanes=-1) == B.ERR_INVALID_ARG
    assert enc(T=-1) == B.ERR_INVALID_ARG
    assert enc(temp=-1.0) == B.ERR_INVALID_ARG
    assert enc(table=None) == B.ERR_INVALID_ARG
    assert enc(prev=None) == B.ERR_INVALID_ARG
    assert enc(seq=None) == B.ERR_INVALID_ARG
    assert enc(lo=None) == B.ERR_INVALID_ARG
    assert enc(lanes=0) == B.OK
    div = lambda **k: L.as_ngram_diversity(k.get("seq", p), p, k.get("S", 1), k.get("N", 2), k.get("T", 4), p, p,
                                           k.get("d", p), None)
    assert div(S=-1) == B.ERR_INVALID_ARG and div(N=0) == B.ERR_INVALID_ARG and div(T=-1) == B.ERR_INVALID_ARG
    assert div(seq=None) == B.ERR_INVALID_ARG and div(d=None) == B.ERR_INVALID_ARG
    assert div(N=32, T=1024) == B.ERR_UNSUPPORTED and div(S=0) == B.OK
    rm = lambda **k: L.as_reward_mean(k.get("seq", p), p, k.get("S", 1), k.get("N", 2), k.get("T", 4), k.get("r", p),
                                      k.get("V", 3), None, k.get("mean", p), None, None)
    assert rm(S=-1) == B.ERR_INVALID_ARG and rm(N=0) == B.ERR_INVALID_ARG and rm(N=5000) == B.ERR_INVALID_ARG
    assert rm(V=0) == B.ERR_INVALID_ARG and rm(r=None) == B.ERR_INVALID_ARG and rm(mean=None) == B.ERR_INVALID_ARG
    assert rm(S=0) == B.OK
    assert L.as_tune(99, 0) == B.ERR_INVALID_ARG and L.as_tune(B.TUNE_CLUSTER, 3) == B.ERR_INVALID_ARG
    assert L.as_tune(B.TUNE_SERIAL_LAUNCH, 2) == B.ERR_INVALID_ARG and L.as_tune(B.TUNE_SERIAL_LAUNCH, 0) == B.OK
    assert L.as_step_host_work_bytes(0, 4, 10) >= 4 * 10 * 4 + 4 * 24


def test_tuning_keys_of_the_binding_match_the_header(L):
    import re
    from paper_2210_15458_b200 import binding as B
    header = open(os.path.join(ROOT, "include", "arith_sampling.h")).read()
    keys = dict(re.findall(r"#define AS_TUNE_(\w+) (\d+)", header))
    assert len(keys) >= 9 and len(set(keys.values())) == len(keys)
    for name, value in keys.items():
        assert getattr(B, "TUNE_" + name) == int(value), name
    assert L.as_tune(B.TUNE_RADIX_NUCLEUS, 2) == B.ERR_INVALID_ARG and L.as_tune(B.TUNE_RADIX_NUCLEUS, 0) == B.OK


def test_no_device_means_an_error_not_a_fallback(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from paper_2210_15458_b200 import binding as B
    buf = (ctypes.c_double * 4)()
    assert L.as_lattice_codes(4, 0.5, ctypes.addressof(buf), None) == B.ERR_CUDA
    assert L.as_last_error() != b""


def test_product_code_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2210_15458_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|oracle/|liboracle", src, flags=re.M), f
