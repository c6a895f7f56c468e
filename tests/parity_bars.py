"""The parity bars of the GPU tests, in one place.

* bf16 attention outputs O: relative-L2 <= 5e-3 and max-abs <= 1e-2, the latter scaled by |value| above 1: the
  bf16 grid's half-spacing is 3.9e-3 at |x| in [1,2), 7.8e-3 at [2,4) and 1.6e-2 at [4,8), so a fixed 1e-2 cannot
  hold for a bf16 number beyond |x| = 2.5, and one dominant key adds 2^-9 |v| from the bf16 probabilities.
* fp32 log-sum-exps: max-abs <= 1e-3, unscaled.  The LSE carries no bf16 rounding (fp32 logits from exact bf16
  products, fp32 row sums of the unrounded probabilities); what remains is the fp32 accumulation of the logits
  (about 1e-6 |s|) and the 2^-22 relative error of ex2.approx, a few 1e-5 at the logit magnitudes tested.
* fp32 response scores (Eq. 2): every element within 1e-3 of its own value plus 1e-6 of the largest score (the
  floor keeps scores that underflow towards zero comparable), and relative-L2 <= 5e-3.  The top-n of Eq. 3 / Eq. 8
  is decided on these values, so no column may be wrong by more than its own rounding.
"""
import numpy as np

MAX_ABS = 1e-2
REL_L2 = 5e-3
LSE_MAX_ABS = 1e-3
SCORE_REL = 1e-3
SCORE_FLOOR = 1e-6

# largest errors seen in this test session (printed in the terminal summary by conftest.py)
WORST = {"O max-abs (scaled)": 0.0, "O rel-L2": 0.0, "lse max-abs": 0.0, "score element error / bound": 0.0,
         "score rel-L2": 0.0}


def _note(key, value):
    WORST[key] = max(WORST[key], float(value))


def np64(x):
    return x.detach().double().cpu().numpy()


def close_o(got, want, what):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    # max-abs 1e-2 for values up to magnitude 1; beyond that the bound scales with the value, because
    # the bf16 output grid itself is coarser than 1e-2 there (half-spacing 2^-7 at |x| in [2,4))
    err = (np.abs(got - want) / np.maximum(1.0, np.abs(want))).max()
    rel = np.linalg.norm((got - want).ravel()) / max(np.linalg.norm(want.ravel()), 1e-30)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    _note("O max-abs (scaled)", err)
    _note("O rel-L2", rel)
    assert err <= MAX_ABS, f"{what}: max-abs (scaled) {err:.3e} > {MAX_ABS}"
    assert rel <= REL_L2, f"{what}: rel-L2 {rel:.3e} > {REL_L2}"


def close_lse(got, want, what):
    """fp32 log-sum-exp against the oracle: plain max-abs, no scaling by the value (a row's normaliser is off
    by the factor exp(err), so 1e-3 nat is a 0.1 % error of the softmax denominator)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    err = np.abs(got - want).max()
    _note("lse max-abs", err)
    assert err <= LSE_MAX_ABS, f"{what}: max-abs {err:.3e} > {LSE_MAX_ABS}"


def close_scores(got, want, what):
    """Response scores (Eq. 2), element by element: |got_i - want_i| <= 1e-3 |want_i| + 1e-6 max|want|."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape and np.isfinite(got).all(), f"{what}: shape or non-finite values"
    bound = SCORE_REL * np.abs(want) + SCORE_FLOOR * np.abs(want).max()
    excess = np.abs(got - want) - bound
    worst = int(np.argmax(excess))
    _note("score element error / bound", (np.abs(got - want) / bound).max())
    assert excess.max() <= 0.0, (f"{what}: element {worst}: got {got.ravel()[worst]:.6e}, want {want.ravel()[worst]:.6e} "
                                 f"({(excess > 0).sum()} elements beyond the bound)")
    rel = np.linalg.norm((got - want).ravel()) / max(np.linalg.norm(want.ravel()), 1e-300)
    _note("score rel-L2", rel)
    assert rel <= REL_L2, f"{what}: rel-L2 {rel:.3e} > {REL_L2}"


