"""ctypes binding of libarith_sampling.so: argument marshalling only.

Every function has the name and argument order of its C entry point
(include/arith_sampling.h); tensors are torch CUDA tensors whose data pointers are
passed through, `stream` defaults to torch's current stream.  bf16 logits may be
torch.bfloat16 tensors or int16/uint16 bit patterns.  There is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import _build

F32 = 0
BF16 = 1
OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_CUDA = -3
ERR_TIMEOUT = -4
ERR_NUMERIC = -5

PATH_COMPACT = 0
PATH_GENERAL = 1

TUNE_STEP_PATH = 1
TUNE_CLUSTER = 2
TUNE_CTAS_PER_SM = 3
TUNE_STAGES = 4
TUNE_MIN_CTAS = 5
TUNE_SERIAL_LAUNCH = 6
TUNE_WAIT_KCYCLES = 7
TUNE_DEBUG_NO_COPY = 8
TUNE_RADIX_NUCLEUS = 9

EXPORTS = ["as_lattice_codes", "as_lattice_codes_variant", "as_step", "as_step_typical", "as_step_lattice", "as_step_host", "as_step_host_work_bytes", "as_step_host_static",
           "as_decode_bigram",
           "as_decode_bigram_codes", "as_xp_lattice_state", "as_decode_bigram_xp", "as_encode_bigram", "as_ngram_diversity", "as_reward_mean", "as_tune",
           "as_last_error", "as_version"]


class AsError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("arith_sampling error %d: %s" % (code, msg))
        self.code = code


class as_step_diag(ctypes.Structure):
    _fields_ = [("d_p_tok", ctypes.c_void_p), ("d_cdf_lo", ctypes.c_void_p),
                ("d_n_kept", ctypes.c_void_p), ("d_lane_status", ctypes.c_void_p),
                ("d_path", ctypes.c_void_p)]


_lib = None


def library_path() -> str:
    return _build.LIB


_path = None


def use_library(path: Optional[str]) -> None:
    """Switch to another build of the library (the bounds-checked one, in tests); None = the default."""
    global _lib, _path
    _lib, _path = None, path


def as_debug_bounds(reset: bool = True):
    """Checked builds only: (failures, first site, its index, its bound) since the last reset."""
    out = (ctypes.c_int * 4)()
    fn = lib().as_debug_bounds
    fn.argtypes = [ctypes.c_void_p, ctypes.c_int]
    fn.restype = ctypes.c_int
    _check(fn(ctypes.cast(out, ctypes.c_void_p), 1 if reset else 0))
    return tuple(out)


def lib():
    """Load the CUDA library (never builds or falls back silently)."""
    global _lib
    if _lib is None:
        path = _path or library_path()
        if not os.path.exists(path):
            raise RuntimeError("CUDA library %s not found: run `python -c 'import __graft_entry__ as g; "
                               "g.build()'` (nvcc, sm_100a) first" % path)
        L = ctypes.CDLL(path)
        P, I, D, LL = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_longlong
        L.as_lattice_codes.argtypes = [I, D, P, P]
        L.as_step.argtypes = [P, I, I, I, LL, P, D, I, D, P, P, ctypes.POINTER(as_step_diag), P]
        L.as_step_typical.argtypes = [P, I, I, I, LL, P, D, I, D, P, P, ctypes.POINTER(as_step_diag), P]
        L.as_step_typical.restype = I
        L.as_step_host.argtypes = [P, I, I, I, LL, P, D, I, D, P, P, P, P, ctypes.c_size_t, P]
        L.as_step_host_static.argtypes = [P, I, I, I, LL, P, D, I, D, P, P, P, P]
        L.as_step_host_static.restype = I
        L.as_step_host_work_bytes.argtypes = [I, I, LL]
        L.as_step_host_work_bytes.restype = ctypes.c_size_t
        L.as_decode_bigram.argtypes = [P, I, I, LL, P, I, I, D, I, I, D, I, D, P, P, P, P, P]
        L.as_decode_bigram_codes.argtypes = [P, I, I, LL, P, P, I, I, I, D, I, D, P, P, P, P, P]
        L.as_encode_bigram.argtypes = [P, I, I, LL, P, P, P, I, I, D, I, D, P, P, P, P]
        L.as_step_lattice.argtypes = [P, I, I, I, LL, I, D, I, D, I, D, P, P, P, P]
        L.as_step_lattice.restype = I
        L.as_lattice_codes_variant.argtypes = [I, D, I, P, P]
        L.as_lattice_codes_variant.restype = I
        L.as_ngram_diversity.argtypes = [P, P, I, I, I, P, P, P, P]
        L.as_reward_mean.argtypes = [P, P, I, I, I, P, I, P, P, P, P]
        L.as_xp_lattice_state.argtypes = [I, D, I, I, I, P, P]
        L.as_xp_lattice_state.restype = I
        L.as_decode_bigram_xp.argtypes = [P, I, I, LL, P, P, I, I, I, I, D, I, D, P, P, P, P]
        L.as_decode_bigram_xp.restype = I
        L.as_tune.argtypes = [I, I]
        L.as_last_error.restype = ctypes.c_char_p
        for n in ("as_lattice_codes", "as_step", "as_step_host", "as_decode_bigram",
                  "as_decode_bigram_codes", "as_xp_lattice_state", "as_decode_bigram_xp", "as_encode_bigram", "as_ngram_diversity", "as_reward_mean", "as_tune",
                  "as_version"):
            getattr(L, n).restype = I
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != OK:
        raise AsError(rc, lib().as_last_error().decode())


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _logits_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype in (torch.bfloat16, torch.int16, torch.uint16):
        return BF16
    raise TypeError("logits must be float32 or bfloat16 (or 16-bit integer bit patterns)")


def _logits_layout(t: torch.Tensor):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("logits / table must be 2-D with unit stride along the vocabulary")
    return t.shape[0], t.shape[1], (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def as_version() -> int:
    return lib().as_version()


def as_tune(key: int, value: int) -> None:
    _check(lib().as_tune(key, value))


def as_lattice_codes(N: int, u: float, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    if out is None:
        out = torch.empty(max(N, 0), dtype=torch.float64, device="cuda")
    _check(lib().as_lattice_codes(N, u, _ptr(out), _stream(stream)))
    return out


LATTICE_SHIFTED, LATTICE_PAPER_DEFINITION, LATTICE_NAIVE = 0, 1, 2
NGRAM_MAX_ITEMS = 16384     # AS_NGRAM_MAX_ITEMS


def as_lattice_codes_variant(N: int, b: float, variant: int, out: Optional[torch.Tensor] = None,
                             stream=None) -> torch.Tensor:
    if out is None:
        out = torch.empty(max(N, 0), dtype=torch.float64, device="cuda")
    _check(lib().as_lattice_codes_variant(N, b, variant, _ptr(out), _stream(stream)))
    return out


def as_step(logits: torch.Tensor, codes: torch.Tensor, temp: float = 1.0, top_k: int = 0,
            top_p: float = 1.0, tokens: Optional[torch.Tensor] = None,
            codes_out: Optional[torch.Tensor] = None, diag: Optional[dict] = None, V: Optional[int] = None,
            stream=None, typical_p: Optional[float] = None):
    """tokens, codes' = one decode step.  `diag`, if a dict, receives the tensors p_tok,
    cdf_lo, n_kept, lane_status, path (allocated here unless already present).  With typical_p
    the call goes to as_step_typical (the typical cut in place of the nucleus)."""
    lanes, width, ld = _logits_layout(logits)
    V = width if V is None else V
    dev = logits.device
    if tokens is None:
        tokens = torch.empty(lanes, dtype=torch.int32, device=dev)
    if codes_out is None:
        codes_out = torch.empty(lanes, dtype=torch.float64, device=dev)
    if codes.dtype != torch.float64 or codes.numel() != lanes:
        raise ValueError("codes must be float64 with one entry per lane")
    dg = None
    if diag is not None:
        diag.setdefault("p_tok", torch.empty(lanes, dtype=torch.float64, device=dev))
        diag.setdefault("cdf_lo", torch.empty(lanes, dtype=torch.float64, device=dev))
        diag.setdefault("n_kept", torch.empty(lanes, dtype=torch.int32, device=dev))
        diag.setdefault("lane_status", torch.empty(lanes, dtype=torch.int32, device=dev))
        diag.setdefault("path", torch.empty(lanes, dtype=torch.int32, device=dev))
        dg = as_step_diag(_ptr(diag["p_tok"]), _ptr(diag["cdf_lo"]), _ptr(diag["n_kept"]),
                          _ptr(diag["lane_status"]), _ptr(diag["path"]))
    if typical_p is not None:
        if 0.0 < top_p < 1.0:
            raise ValueError("a step takes top_p or typical_p, not both")
        _check(lib().as_step_typical(_ptr(logits), _logits_dtype(logits), lanes, V, ld, _ptr(codes), temp, top_k,
                                     typical_p, _ptr(tokens), _ptr(codes_out),
                                     ctypes.byref(dg) if dg is not None else None, _stream(stream)))
        return tokens, codes_out
    _check(lib().as_step(_ptr(logits), _logits_dtype(logits), lanes, V, ld, _ptr(codes), temp, top_k, top_p,
                         _ptr(tokens), _ptr(codes_out), ctypes.byref(dg) if dg is not None else None,
                         _stream(stream)))
    return tokens, codes_out


def as_step_lattice(logits: torch.Tensor, N: int, u: float, j0: int = 0, temp: float = 1.0, top_k: int = 0,
                    top_p: float = 1.0, tokens: Optional[torch.Tensor] = None,
                    codes_out: Optional[torch.Tensor] = None, V: Optional[int] = None, stream=None):
    """First decode step with the lattice codes (j0 + i + u)/N formed in the kernel."""
    lanes, width, ld = _logits_layout(logits)
    V = width if V is None else V
    dev = logits.device
    if tokens is None:
        tokens = torch.empty(lanes, dtype=torch.int32, device=dev)
    if codes_out is None:
        codes_out = torch.empty(lanes, dtype=torch.float64, device=dev)
    _check(lib().as_step_lattice(_ptr(logits), _logits_dtype(logits), lanes, V, ld, N, u, j0, temp, top_k, top_p,
                                 _ptr(tokens), _ptr(codes_out), None, _stream(stream)))
    return tokens, codes_out


def as_step_host_work_bytes(dtype: int, lanes: int, ld: int) -> int:
    return lib().as_step_host_work_bytes(dtype, lanes, ld)


def as_step_host(h_logits: torch.Tensor, h_codes: torch.Tensor, temp: float, top_k: int, top_p: float,
                 h_tokens: torch.Tensor, h_codes_out: torch.Tensor, h_lane_status: Optional[torch.Tensor],
                 d_work: torch.Tensor, V: Optional[int] = None, stream=None) -> None:
    """Host-buffer step: all h_* are CPU tensors (pinned for speed), d_work a CUDA byte buffer."""
    lanes, width, ld = _logits_layout(h_logits)
    V = width if V is None else V
    _check(lib().as_step_host(_ptr(h_logits), _logits_dtype(h_logits), lanes, V, ld, _ptr(h_codes), temp,
                              top_k, top_p, _ptr(h_tokens), _ptr(h_codes_out), _ptr(h_lane_status),
                              _ptr(d_work), d_work.numel() * d_work.element_size(), _stream(stream)))


STATIC_WORK_BYTES = 24 << 20


def as_step_host_static(h_logits: torch.Tensor, h_codes: torch.Tensor, temp: float, top_k: int, top_p: float,
                        h_tokens: torch.Tensor, h_codes_out: torch.Tensor, h_lane_status: Optional[torch.Tensor],
                        V: Optional[int] = None, stream=None) -> None:
    """as_step_host for callers that own no device memory: the device work space is a buffer
    built into the library (STATIC_WORK_BYTES).  Every tensor here is a CPU tensor; nothing is
    allocated on the device, neither by the library nor by this wrapper.  Steps that need more
    work space than the buffer holds raise AsError(ERR_UNSUPPORTED).  Calls share the buffer, so
    do not let two of them overlap on the GPU."""
    lanes, width, ld = _logits_layout(h_logits)
    V = width if V is None else V
    _check(lib().as_step_host_static(_ptr(h_logits), _logits_dtype(h_logits), lanes, V, ld, _ptr(h_codes), temp,
                                     top_k, top_p, _ptr(h_tokens), _ptr(h_codes_out), _ptr(h_lane_status),
                                     _stream(stream)))


def as_decode_bigram(table: torch.Tensor, start_tokens: torch.Tensor, N: int, u: float, T: int, eos: int,
                     temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None,
                     codes_final: Optional[torch.Tensor] = None, lane_status: Optional[torch.Tensor] = None,
                     seq: Optional[torch.Tensor] = None, length: Optional[torch.Tensor] = None, stream=None,
                     per_step: bool = True):
    rows, width, ld = _logits_layout(table)
    V = width if V is None else V
    if rows < V:
        raise ValueError("bigram table needs at least V rows")
    S = start_tokens.numel()
    lanes = S * max(N, 0)
    dev = table.device
    if codes_final is None and per_step:    # also the loop's state for the per-step kernels
        codes_final = torch.empty(lanes, dtype=torch.float64, device=dev)
    if seq is None:
        seq = torch.empty((lanes, T), dtype=torch.int32, device=dev)
    if length is None:
        length = torch.empty(lanes, dtype=torch.int32, device=dev)
    _check(lib().as_decode_bigram(_ptr(table), _logits_dtype(table), V, ld, _ptr(start_tokens), S, N, u, T, eos,
                                  temp, top_k, top_p, _ptr(seq), _ptr(length), _ptr(codes_final),
                                  _ptr(lane_status), _stream(stream)))
    return seq, length


def as_decode_bigram_codes(table: torch.Tensor, prev: torch.Tensor, codes_in: torch.Tensor, T: int, eos: int,
                           temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None,
                           codes_final: Optional[torch.Tensor] = None,
                           lane_status: Optional[torch.Tensor] = None, seq: Optional[torch.Tensor] = None,
                           length: Optional[torch.Tensor] = None, stream=None, per_step: bool = True):
    rows, width, ld = _logits_layout(table)
    V = width if V is None else V
    if rows < V:
        raise ValueError("bigram table needs at least V rows")
    lanes = prev.numel()
    dev = table.device
    if codes_final is None and per_step:    # also the loop's state for the per-step kernels
        codes_final = torch.empty(lanes, dtype=torch.float64, device=dev)
    if seq is None:
        seq = torch.empty((lanes, T), dtype=torch.int32, device=dev)
    if length is None:
        length = torch.empty(lanes, dtype=torch.int32, device=dev)
    _check(lib().as_decode_bigram_codes(_ptr(table), _logits_dtype(table), V, ld, _ptr(prev), _ptr(codes_in),
                                        lanes, T, eos, temp, top_k, top_p, _ptr(seq), _ptr(length),
                                        _ptr(codes_final), _ptr(lane_status), _stream(stream)))
    return seq, length


def as_xp_lattice_state(N: int, u: float, j0: int = 0, count: Optional[int] = None, S: int = 1,
                        out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """int64 [S*count, 4] (the bits of four unsigned 64-bit words per lane): decoder state of the
    lattice codes (j + u)/N, j = j0 .. j0+count-1, one copy per start token."""
    count = N - j0 if count is None else count
    if out is None:
        out = torch.empty((max(S, 0) * max(count, 0), 4), dtype=torch.int64, device="cuda")
    _check(lib().as_xp_lattice_state(N, u, j0, count, S, _ptr(out), _stream(stream)))
    return out


def as_decode_bigram_xp(table: torch.Tensor, prev: torch.Tensor, state: torch.Tensor, N: int, T: int, eos: int,
                        temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None,
                        lane_status: Optional[torch.Tensor] = None, seq: Optional[torch.Tensor] = None,
                        length: Optional[torch.Tensor] = None, stream=None):
    """Algorithm 1's loop with extended-precision codes; `state` [lanes, 4] int64 is updated in place."""
    rows, width, ld = _logits_layout(table)
    V = width if V is None else V
    if rows < V:
        raise ValueError("bigram table needs at least V rows")
    lanes = prev.numel()
    if state.dtype != torch.int64 or state.numel() != 4 * lanes or not state.is_contiguous():
        raise ValueError("state must be a contiguous [lanes, 4] int64 tensor")
    dev = table.device
    if seq is None:
        seq = torch.empty((lanes, T), dtype=torch.int32, device=dev)
    if length is None:
        length = torch.empty(lanes, dtype=torch.int32, device=dev)
    _check(lib().as_decode_bigram_xp(_ptr(table), _logits_dtype(table), V, ld, _ptr(prev), _ptr(state), lanes, N, T,
                                     eos, temp, top_k, top_p, _ptr(seq), _ptr(length), _ptr(lane_status),
                                     _stream(stream)))
    return seq, length


def as_encode_bigram(table: torch.Tensor, prev: torch.Tensor, seq: torch.Tensor, length: torch.Tensor,
                     temp: float = 1.0, top_k: int = 0, top_p: float = 1.0, V: Optional[int] = None,
                     lane_status: Optional[torch.Tensor] = None, stream=None):
    """Interval [lo, lo + width) of each lane's sequence in dictionary order (Sec. 4.1)."""
    rows, width_, ld = _logits_layout(table)
    V = width_ if V is None else V
    if rows < V:
        raise ValueError("bigram table needs at least V rows")
    if seq.dim() != 2 or not seq.is_contiguous() or seq.dtype != torch.int32:
        raise ValueError("seq must be a contiguous [lanes, T] int32 tensor")
    lanes, T = seq.shape
    if prev.numel() != lanes or length.numel() != lanes:
        raise ValueError("prev and length need one entry per lane")
    dev = table.device
    lo = torch.empty(lanes, dtype=torch.float64, device=dev)
    width = torch.empty(lanes, dtype=torch.float64, device=dev)
    _check(lib().as_encode_bigram(_ptr(table), _logits_dtype(table), V, ld, _ptr(prev), _ptr(seq), _ptr(length),
                                  lanes, T, temp, top_k, top_p, _ptr(lo), _ptr(width), _ptr(lane_status),
                                  _stream(stream)))
    return lo, width


def _groups(seq: torch.Tensor, length: torch.Tensor, N: int):
    if seq.dim() != 2 or not seq.is_contiguous() or seq.dtype != torch.int32:
        raise ValueError("seq must be a contiguous [lanes, T] int32 tensor")
    lanes, T = seq.shape
    if N < 1 or lanes % N or length.numel() != lanes:
        raise ValueError("lanes must be a multiple of N, with one length per lane")
    return lanes // N, T


def as_ngram_diversity(seq: torch.Tensor, length: torch.Tensor, N: int, stream=None):
    """(unique[S,4], total[S,4], d[S]): n-gram diversity of each group of N lanes (Sec. 5.1)."""
    S, T = _groups(seq, length, N)
    dev = seq.device
    unique = torch.empty((S, 4), dtype=torch.int64, device=dev)
    total = torch.empty((S, 4), dtype=torch.int64, device=dev)
    d = torch.empty(S, dtype=torch.float64, device=dev)
    _check(lib().as_ngram_diversity(_ptr(seq), _ptr(length), S, N, T, _ptr(unique), _ptr(total), _ptr(d),
                                    _stream(stream)))
    return unique, total, d


def as_reward_mean(seq: torch.Tensor, length: torch.Tensor, N: int, r: torch.Tensor,
                   group_status: Optional[torch.Tensor] = None, stream=None):
    """(lane_reward[lanes], mean[S]) for the additive reward r[token] (Sec. 4.2 estimator)."""
    S, T = _groups(seq, length, N)
    if r.dtype != torch.float64 or not r.is_contiguous():
        raise ValueError("r must be a contiguous float64 tensor")
    dev = seq.device
    lane_reward = torch.empty(S * N, dtype=torch.float64, device=dev)
    mean = torch.empty(S, dtype=torch.float64, device=dev)
    _check(lib().as_reward_mean(_ptr(seq), _ptr(length), S, N, T, _ptr(r), r.numel(), _ptr(lane_reward),
                                _ptr(mean), _ptr(group_status), _stream(stream)))
    return lane_reward, mean
