import numpy as np

from tests.helpers import rel_errors


def test_rel_error_metric_sanity():
    ref = np.array([[1.0, -2.0], [0.5, 0.25]])
    got = ref + np.array([[0.0, 0.02], [0.0, 0.0]])
    emax, emean = rel_errors(got, ref)
    assert np.isclose(emax, 0.01) and np.isclose(emean, (0.02 / 3.0) / 2)
