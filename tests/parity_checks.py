"""Checks shared by the GPU parity tests (no arithmetic of the method: comparisons only)."""
import numpy as np


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def assert_expert_counts(counts_gpu, logw_ref, margin=1e-4):
    """n_alpha of Eq. 10 (how many positions have expert alpha as their largest gate weight) is integer
    work, so the bar is exact.  The library takes the argmax of its fp32 gate logits; where the oracle's two
    largest log-weights of a position differ by more than `margin` (far above fp32 rounding of a d-term dot
    product) both sides must name the same expert.  Positions inside the margin (there must be almost none)
    may go to either, which widens the admissible range of an expert's count by exactly their number."""
    logw = np.asarray(logw_ref, dtype=np.float64)
    got = np.asarray(counts_gpu, dtype=np.int64)
    N, r = logw.shape
    assert got.shape == (r,)
    assert int(got.sum()) == N
    if r == 1:
        assert int(got[0]) == N
        return
    ordered = np.sort(logw, axis=1)
    clear = (ordered[:, -1] - ordered[:, -2]) > margin
    ambiguous = int(N - clear.sum())
    assert ambiguous <= 0.01 * N, f"{ambiguous} of {N} positions have a gate margin below {margin}"
    ref_clear = np.bincount(np.argmax(logw[clear], axis=1), minlength=r).astype(np.int64)
    assert np.all(got >= ref_clear), (got, ref_clear)
    assert np.all(got - ref_clear <= ambiguous), (got, ref_clear, ambiguous)
    if ambiguous == 0:
        assert np.array_equal(got, ref_clear)
