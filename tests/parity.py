"""Shared comparison of a CUDA step result with the oracle's (tolerances in one place).

Tokens must match exactly wherever the oracle's code lies more than TOK_BAND from a CDF
boundary and the nucleus cut is more than TOPP_BAND from the target mass; inside those
bands several answers are correct in floating point, so such lanes are only counted.
On the compared lanes the rescaled code must agree to CODE_RTOL and the chosen token's
probability to PTOK_RTOL (relative).
"""
import numpy as np

TOK_BAND = 1e-5
TOPP_BAND = 1e-6
CODE_RTOL = 1e-6
PTOK_RTOL = 1e-5


def compare_step(ref, tokens, codes, p_tok=None, n_kept=None, status=None, what=""):
    tokens = np.asarray(tokens)
    codes = np.asarray(codes)
    ok = ref.status == 0
    if status is not None:
        np.testing.assert_array_equal(np.asarray(status), ref.status, err_msg=what + " lane status")
        bad = ~ok
        assert (tokens[bad] == -1).all(), what + " failed lanes must return token -1"
    safe = ok & (ref.d_tok > TOK_BAND) & (ref.d_topp > TOPP_BAND)
    mism = np.nonzero(safe & (tokens != ref.tokens))[0]
    assert mism.size == 0, "%s token mismatch on lanes %s: got %s want %s (d_tok %s)" % (
        what, mism[:8], tokens[mism[:8]], ref.tokens[mism[:8]], ref.d_tok[mism[:8]])
    np.testing.assert_allclose(codes[safe], ref.codes[safe], rtol=CODE_RTOL, atol=1e-12,
                               err_msg=what + " rescaled code")
    if p_tok is not None:
        np.testing.assert_allclose(np.asarray(p_tok)[safe], ref.p_tok[safe], rtol=PTOK_RTOL,
                                   err_msg=what + " p_tok")
    if n_kept is not None:
        sel = ok & (ref.d_topp > TOPP_BAND)
        np.testing.assert_array_equal(np.asarray(n_kept)[sel], ref.n_kept[sel], err_msg=what + " n_kept")
    unsafe = ok & ~safe
    return {"lanes": int(ok.size), "compared": int(safe.sum()), "near_boundary": int(unsafe.sum()),
            "near_boundary_token_diff": int((tokens[unsafe] != ref.tokens[unsafe]).sum())}
