"""The parity comparator itself (CPU only): what it must reject."""
import numpy as np
import pytest
import torch

from helpers import assert_within_bound


def test_comparator_accepts_values_inside_the_bound():
    want = np.array([[1.0, -2.0], [0.5, 0.0]])
    S = np.array([[10.0, 10.0], [10.0, 10.0]])
    got = torch.tensor(want + 5e-4)              # bound is 1e-3
    assert assert_within_bound(got, want, S) == pytest.approx(5e-5)


def test_comparator_rejects_values_outside_the_bound():
    want = np.zeros((2, 2))
    S = np.ones((2, 2))
    got = torch.zeros(2, 2, dtype=torch.float64)
    got[1, 0] = 2e-4
    with pytest.raises(AssertionError, match="1 of 4 elements outside"):
        assert_within_bound(got, want, S)


@pytest.mark.parametrize("value", [float("nan"), float("inf"), -float("inf")])
def test_comparator_rejects_unwritten_or_non_finite_elements(value):
    # overwrite-mode tests fill the output with NaN before the call: an element the kernel never wrote must fail
    want = np.zeros((3, 3))
    S = np.ones((3, 3))
    got = torch.zeros(3, 3)
    got[2, 1] = value
    with pytest.raises(AssertionError, match="NaN or infinite"):
        assert_within_bound(got, want, S)


def test_comparator_rejects_a_nan_in_the_expectation_or_the_scale():
    got = torch.zeros(2)
    with pytest.raises(AssertionError):
        assert_within_bound(got, np.array([0.0, np.nan]), np.ones(2))
    with pytest.raises(AssertionError):
        assert_within_bound(got, np.zeros(2), np.array([1.0, np.nan]))


def test_comparator_checks_shapes():
    with pytest.raises(AssertionError):
        assert_within_bound(torch.zeros(2, 3), np.zeros((3, 2)), np.ones((3, 2)))
