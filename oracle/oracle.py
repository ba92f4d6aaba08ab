"""ctypes binding of the CPU oracle (oracle/as_oracle.c) -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.
It never touches the CUDA library.  `build()` compiles the C file with gcc into
oracle/liboracle.so (rebuilt when the source is newer).

Arrays: fp32 logits are numpy float32, bf16 logits are numpy uint16 bit
patterns; codes are float64; tokens int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "as_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32 = 0
BF16 = 1
OK = 0
ERR_INVALID_ARG = -1
ERR_NUMERIC = -5

_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        L = ctypes.c_long
        D = ctypes.c_double
        P = ctypes.c_void_p
        _lib.orc_lattice_codes.argtypes = [L, D, P]
        _lib.orc_step.argtypes = [P, ctypes.c_int, L, L, L, P, D, L, D] + [P] * 9 + [L, L]
        _lib.orc_step_typical.argtypes = [P, ctypes.c_int, L, L, L, P, D, L, D] + [P] * 9 + [L, L]
        _lib.orc_step_typical.restype = ctypes.c_int
        _lib.orc_decode_bigram_codes.argtypes = ([P, ctypes.c_int, L, L, P, P, L, L, L, D, L, D]
                                                 + [P] * 8 + [L, L])
        _lib.orc_decode_bigram.argtypes = [P, ctypes.c_int, L, L, P, L, L, D, L, L, D, L, D, P, P, P, P]
        _lib.orc_encode_bigram.argtypes = [P, ctypes.c_int, L, L, P, P, P, L, L, D, L, D, P, P, P]
        _lib.orc_lattice_codes_variant.argtypes = [L, D, L, P]
        _lib.orc_lattice_codes_variant.restype = ctypes.c_int
        _lib.orc_ngram_diversity.argtypes = [P, P, L, L, L, P, P, P]
        _lib.orc_reward_mean.argtypes = [P, P, L, L, L, P, L, P, P]
        _lib.orc_xp_lattice_state.argtypes = [L, D, L, L, L, P]
        _lib.orc_xp_row_cells.argtypes = [P, ctypes.c_int, L, D, L, D, P]
        _lib.orc_xp_decode_bigram.argtypes = [P, ctypes.c_int, L, L, P, P, L, L, L, L, D, L, D, P, P, P, P, P, L, L]
        for f in (_lib.orc_xp_lattice_state, _lib.orc_xp_row_cells, _lib.orc_xp_decode_bigram):
            f.restype = ctypes.c_int
        for f in (_lib.orc_lattice_codes, _lib.orc_step, _lib.orc_decode_bigram_codes,
                  _lib.orc_decode_bigram, _lib.orc_encode_bigram, _lib.orc_ngram_diversity,
                  _lib.orc_reward_mean, _lib.orc_version):
            f.restype = ctypes.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_logits(a: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == F32 else np.uint16
    if a.dtype != want or a.ndim != 2 or not a.flags.c_contiguous:
        raise ValueError("logits must be a C-contiguous 2-D %s array" % want.__name__)
    return a


def _ranges(n: int, threads: int):
    threads = max(1, min(threads, n if n > 0 else 1))
    edges = np.linspace(0, n, threads + 1).astype(np.int64)
    return [(int(edges[i]), int(edges[i + 1])) for i in range(threads) if edges[i + 1] > edges[i]]


def _run_ranges(fn, n: int, threads: int) -> None:
    rs = _ranges(n, threads)
    if len(rs) <= 1:
        for a, b in rs:
            rc = fn(a, b)
            if rc != OK:
                raise ValueError("oracle returned %d" % rc)
        return
    with ThreadPoolExecutor(len(rs)) as ex:   # ctypes releases the GIL; lanes are independent
        for rc in ex.map(lambda ab: fn(*ab), rs):
            if rc != OK:
                raise ValueError("oracle returned %d" % rc)


def lattice_codes(N: int, u: float) -> np.ndarray:
    out = np.empty(max(N, 0), dtype=np.float64)
    rc = lib().orc_lattice_codes(N, u, _ptr(out))
    if rc != OK:
        raise ValueError("orc_lattice_codes: invalid argument")
    return out


def lattice_codes_variant(N: int, b: float, variant: int) -> np.ndarray:
    """variant 0: (j+b)/N; 1: (i/(N+1) + b) mod 1; 2: i/(N+1) (no shift)."""
    out = np.empty(max(N, 0), dtype=np.float64)
    rc = lib().orc_lattice_codes_variant(N, b, variant, _ptr(out))
    if rc != OK:
        raise ValueError("orc_lattice_codes_variant: invalid argument")
    return out


@dataclass
class StepOut:
    tokens: np.ndarray
    codes: np.ndarray
    p_tok: np.ndarray
    cdf_lo: np.ndarray
    n_kept: np.ndarray
    d_tok: np.ndarray
    d_topp: np.ndarray
    tie_topk: np.ndarray
    status: np.ndarray


def step(logits: np.ndarray, dtype: int, codes: np.ndarray, temp: float = 1.0, top_k: int = 0,
         top_p: float = 1.0, V: Optional[int] = None, threads: int = 1, typical_p: float = 1.0) -> StepOut:
    """One decode step per lane.  typical_p in (0,1): the locally typical cut instead of the nucleus."""
    typical = 0.0 < typical_p < 1.0
    if typical and 0.0 < top_p < 1.0:
        raise ValueError("a step takes a nucleus or a typical cut, not both")
    fn = lib().orc_step_typical if typical else lib().orc_step
    cutp = typical_p if typical else top_p
    logits = _check_logits(logits, dtype)
    lanes, ld = logits.shape
    V = ld if V is None else V
    codes = np.ascontiguousarray(codes, dtype=np.float64)
    if codes.shape != (lanes,):
        raise ValueError("codes must have one entry per lane")
    o = StepOut(np.empty(lanes, np.int32), np.empty(lanes, np.float64), np.empty(lanes, np.float64),
                np.empty(lanes, np.float64), np.empty(lanes, np.int32), np.empty(lanes, np.float64),
                np.empty(lanes, np.float64), np.empty(lanes, np.int32), np.empty(lanes, np.int32))

    def run(a, b):
        return fn(_ptr(logits), dtype, lanes, V, ld, _ptr(codes), temp, top_k, cutp,
                              _ptr(o.tokens), _ptr(o.codes), _ptr(o.p_tok), _ptr(o.cdf_lo),
                              _ptr(o.n_kept), _ptr(o.d_tok), _ptr(o.d_topp), _ptr(o.tie_topk),
                              _ptr(o.status), a, b)
    if lanes == 0:
        if lib().orc_step(_ptr(logits), dtype, 0, V, ld, _ptr(codes), temp, top_k, top_p,
                          *([None] * 9), 0, 0) != OK:
            raise ValueError("oracle returned invalid argument")
        return o
    _run_ranges(run, lanes, threads)
    return o


@dataclass
class DecodeOut:
    seq: np.ndarray
    len: np.ndarray
    codes_final: np.ndarray
    status: np.ndarray
    trace_code_in: Optional[np.ndarray] = None
    trace_code_out: Optional[np.ndarray] = None
    trace_p_tok: Optional[np.ndarray] = None
    trace_d_tok: Optional[np.ndarray] = None


def decode_bigram_codes(table: np.ndarray, dtype: int, prev: np.ndarray, codes: np.ndarray, T: int,
                        eos: int, temp: float = 1.0, top_k: int = 0, top_p: float = 1.0,
                        V: Optional[int] = None, trace: bool = False, threads: int = 1) -> DecodeOut:
    table = _check_logits(table, dtype)
    ld = table.shape[1]
    V = ld if V is None else V
    prev = np.ascontiguousarray(prev, dtype=np.int32)
    codes = np.ascontiguousarray(codes, dtype=np.float64)
    lanes = prev.shape[0]
    if codes.shape != (lanes,):
        raise ValueError("codes and prev must have one entry per lane")
    if lanes and (prev.min() < 0 or prev.max() >= min(V, table.shape[0])):
        raise ValueError("prev token out of range")
    o = DecodeOut(np.empty((lanes, T), np.int32), np.empty(lanes, np.int32),
                  np.empty(lanes, np.float64), np.empty(lanes, np.int32))
    if trace:
        o.trace_code_in = np.empty((lanes, T), np.float64)
        o.trace_code_out = np.empty((lanes, T), np.float64)
        o.trace_p_tok = np.empty((lanes, T), np.float64)
        o.trace_d_tok = np.empty((lanes, T), np.float64)

    def run(a, b):
        return lib().orc_decode_bigram_codes(
            _ptr(table), dtype, V, ld, _ptr(prev), _ptr(codes), lanes, T, eos, temp, top_k, top_p,
            _ptr(o.seq), _ptr(o.len), _ptr(o.codes_final), _ptr(o.status), _ptr(o.trace_code_in),
            _ptr(o.trace_code_out), _ptr(o.trace_p_tok), _ptr(o.trace_d_tok), a, b)
    _run_ranges(run, lanes, threads)
    return o


def decode_bigram(table: np.ndarray, dtype: int, start: np.ndarray, N: int, u: float, T: int, eos: int,
                  temp: float = 1.0, top_k: int = 0, top_p: float = 1.0,
                  V: Optional[int] = None) -> DecodeOut:
    table = _check_logits(table, dtype)
    ld = table.shape[1]
    V = ld if V is None else V
    start = np.ascontiguousarray(start, dtype=np.int32)
    S = start.shape[0]
    if S and (start.min() < 0 or start.max() >= min(V, table.shape[0])):
        raise ValueError("start token out of range")
    lanes = S * max(N, 0)
    o = DecodeOut(np.empty((lanes, T), np.int32), np.empty(lanes, np.int32),
                  np.empty(lanes, np.float64), np.empty(lanes, np.int32))
    rc = lib().orc_decode_bigram(_ptr(table), dtype, V, ld, _ptr(start), S, N, u, T, eos, temp,
                                 top_k, top_p, _ptr(o.seq), _ptr(o.len), _ptr(o.codes_final),
                                 _ptr(o.status))
    if rc != OK:
        raise ValueError("orc_decode_bigram returned %d" % rc)
    return o


def encode_bigram(table: np.ndarray, dtype: int, prev: np.ndarray, seq: np.ndarray, length: np.ndarray,
                  temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None):
    """Interval [lo, lo+width) of each lane's sequence in dictionary order."""
    table = _check_logits(table, dtype)
    ld = table.shape[1]
    V = ld if V is None else V
    prev = np.ascontiguousarray(prev, dtype=np.int32)
    seq = np.ascontiguousarray(seq, dtype=np.int32)
    length = np.ascontiguousarray(length, dtype=np.int32)
    lanes, T = seq.shape
    lo = np.empty(lanes, np.float64)
    width = np.empty(lanes, np.float64)
    status = np.empty(lanes, np.int32)
    rc = lib().orc_encode_bigram(_ptr(table), dtype, V, ld, _ptr(prev), _ptr(seq), _ptr(length), lanes, T,
                                 temp, top_k, top_p, _ptr(lo), _ptr(width), _ptr(status))
    if rc != OK:
        raise ValueError("orc_encode_bigram returned %d" % rc)
    return lo, width, status


def ngram_diversity(seq: np.ndarray, length: np.ndarray, N: int):
    """(unique[S,4], total[S,4], d[S]) of Sec. 5.1's n-gram diversity per group of N lanes."""
    seq = np.ascontiguousarray(seq, dtype=np.int32)
    length = np.ascontiguousarray(length, dtype=np.int32)
    lanes, T = seq.shape
    if lanes % N:
        raise ValueError("lanes must be a multiple of N")
    S = lanes // N
    unique = np.empty((S, 4), np.int64)
    total = np.empty((S, 4), np.int64)
    d = np.empty(S, np.float64)
    rc = lib().orc_ngram_diversity(_ptr(seq), _ptr(length), S, N, T, _ptr(unique), _ptr(total), _ptr(d))
    if rc != OK:
        raise ValueError("orc_ngram_diversity returned %d" % rc)
    return unique, total, d


def reward_mean(seq: np.ndarray, length: np.ndarray, N: int, r: np.ndarray):
    """(lane_reward[lanes], mean[S]): additive reward per lane and its mean per group of N lanes."""
    seq = np.ascontiguousarray(seq, dtype=np.int32)
    length = np.ascontiguousarray(length, dtype=np.int32)
    r = np.ascontiguousarray(r, dtype=np.float64)
    lanes, T = seq.shape
    if lanes % N:
        raise ValueError("lanes must be a multiple of N")
    S = lanes // N
    lane_reward = np.empty(lanes, np.float64)
    mean = np.empty(S, np.float64)
    rc = lib().orc_reward_mean(_ptr(seq), _ptr(length), S, N, T, _ptr(r), len(r), _ptr(lane_reward), _ptr(mean))
    if rc != OK:
        raise ValueError("orc_reward_mean returned %d" % rc)
    return lane_reward, mean


# ----------------------------------------------------------------------------- extended-precision codes
def xp_lattice_state(N: int, u: float, S: int = 1, j0: int = 0, count: Optional[int] = None) -> np.ndarray:
    """uint64 [S*count, 4]: decoder state of the lattice codes (j + floor(u 2^53)/2^53)/N for
    j = j0 .. j0+count-1 (default: all N), one copy per start token."""
    count = N - j0 if count is None else count
    out = np.zeros((max(S, 0) * max(count, 0), 4), dtype=np.uint64)
    rc = lib().orc_xp_lattice_state(N, u, j0, count, S, _ptr(out))
    if rc != OK:
        raise ValueError("orc_xp_lattice_state: invalid argument")
    return out


def xp_row_cells(row: np.ndarray, dtype: int, temp: float = 1.0, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """uint64 [V+1]: the 2^32-cell boundaries F(P_j) of one row's modified distribution."""
    row = np.ascontiguousarray(row)
    V = row.shape[0]
    cells = np.zeros(V + 1, dtype=np.uint64)
    rc = lib().orc_xp_row_cells(_ptr(row), dtype, V, temp, top_k, top_p, _ptr(cells))
    if rc != OK:
        raise ValueError("orc_xp_row_cells returned %d" % rc)
    return cells


@dataclass
class XpDecodeOut:
    seq: np.ndarray
    len: np.ndarray
    status: np.ndarray
    state: np.ndarray
    trace_pos: Optional[np.ndarray] = None
    trace_d_tok: Optional[np.ndarray] = None


def xp_decode_bigram(table: np.ndarray, dtype: int, prev: np.ndarray, state: np.ndarray, N: int, T: int, eos: int,
                     temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None,
                     trace: bool = False, threads: int = 1) -> XpDecodeOut:
    """Algorithm 1's loop with extended-precision codes; `state` [lanes, 4] uint64 is not modified
    (the updated copy is returned)."""
    table = _check_logits(table, dtype)
    ld = table.shape[1]
    V = ld if V is None else V
    prev = np.ascontiguousarray(prev, dtype=np.int32)
    state = np.array(state, dtype=np.uint64, copy=True)
    lanes = prev.shape[0]
    if state.shape != (lanes, 4):
        raise ValueError("state must be [lanes, 4] uint64")
    o = XpDecodeOut(np.empty((lanes, T), np.int32), np.empty(lanes, np.int32), np.empty(lanes, np.int32), state)
    if trace:
        o.trace_pos = np.empty((lanes, T), np.float64)
        o.trace_d_tok = np.empty((lanes, T), np.float64)

    def run(a, b):
        return lib().orc_xp_decode_bigram(_ptr(table), dtype, V, ld, _ptr(prev), _ptr(state), lanes, N, T, eos, temp,
                                          top_k, top_p, _ptr(o.seq), _ptr(o.len), _ptr(o.status),
                                          _ptr(o.trace_pos), _ptr(o.trace_d_tok), a, b)
    _run_ranges(run, lanes, threads)
    return o
