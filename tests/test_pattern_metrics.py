"""Host-side pattern comparison helpers against hand-counted cases."""
import numpy as np

from paper_2509_24014_b200 import pattern_metrics as pm


def test_recall_and_mass_on_a_hand_counted_case():
    nb = 6
    # rows: {0,2,5}, {1}, {} (empty), {3,4}
    ref_rp = np.array([0, 3, 4, 4, 6], dtype=np.int32)
    ref_ci = np.array([0, 2, 5, 1, 3, 4], dtype=np.int32)
    # rows: {0,5}, {2}, {1}, {3,4,5}
    rp = np.array([0, 2, 3, 4, 7], dtype=np.int32)
    ci = np.array([0, 5, 2, 1, 3, 4, 5], dtype=np.int32)
    np.testing.assert_allclose(pm.pattern_recall(ref_rp, ref_ci, rp, ci, nb), [2 / 3, 0.0, 1.0, 1.0])
    np.testing.assert_allclose(pm.pattern_recall(ref_rp, ref_ci, ref_rp, ref_ci, nb), 1.0)
    scores = np.arange(24, dtype=np.float32).reshape(4, 6)
    np.testing.assert_allclose(pm.kept_mass(scores, ref_rp, ref_ci), [0 + 2 + 5, 7, 0, 21 + 22])
    np.testing.assert_allclose(pm.kept_mass(scores, rp, ci), [0 + 5, 8, 13, 21 + 22 + 23])


def test_capacity_padding_after_nnz_is_ignored():
    rp = np.array([0, 1, 2], dtype=np.int32)
    ci = np.array([1, 0, 7, 7, 7], dtype=np.int32)   # entries past row_ptr[-1] are unused capacity
    np.testing.assert_allclose(pm.pattern_recall(rp, ci, rp, ci[:2], 4), 1.0)
