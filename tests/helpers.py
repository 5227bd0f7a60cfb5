"""Shared test helpers: tolerances of the parity bar and small wrappers."""
import numpy as np

from paper_2604_18655_b200.runtime import MloraModel as GpuModel  # noqa: F401  (re-exported for tests)

# parity bar for floating-point outputs against the oracle
MAX_ABS_FRAC = 1e-2      # max|d| <= 1e-2 * max|ref|
REL_L2 = 5e-3            # ||d||_2 <= 5e-3 * ||ref||_2
ARGMAX_MARGIN = 1e-2     # tokens must agree wherever the oracle's top-2 logit gap exceeds this


def compare(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    d = got - want
    max_abs, ref_max = np.abs(d).max(), np.abs(want).max()
    rel_l2 = np.linalg.norm(d) / max(np.linalg.norm(want), 1e-30)
    assert max_abs <= MAX_ABS_FRAC * ref_max, f"{what}: max|d| {max_abs:.3e} > {MAX_ABS_FRAC} * {ref_max:.3e}"
    assert rel_l2 <= REL_L2, f"{what}: rel-L2 {rel_l2:.3e} > {REL_L2}"
    return max_abs / max(ref_max, 1e-30), rel_l2


def check_argmax(gpu_tokens, oracle_logits, what=""):
    """GPU greedy tokens must equal the oracle's argmax wherever the oracle's top-2 margin is decisive."""
    gpu_tokens = np.asarray(gpu_tokens).reshape(-1)
    lg = np.asarray(oracle_logits, dtype=np.float64).reshape(len(gpu_tokens), -1)
    part = np.partition(lg, -2, axis=1)
    margin = part[:, -1] - part[:, -2]
    am = np.argmax(lg, axis=1)
    n_ties = 0
    for i, (g, a) in enumerate(zip(gpu_tokens, am)):
        if g != a:
            assert margin[i] <= ARGMAX_MARGIN, f"{what}: row {i} token {g} != oracle {a} with margin {margin[i]:.4f}"
            # the GPU's choice must itself be a near-maximum
            assert lg[i, a] - lg[i, g] <= ARGMAX_MARGIN, f"{what}: row {i} picked a non-maximal token"
            n_ties += 1
    return n_ties
