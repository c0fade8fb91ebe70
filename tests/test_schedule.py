"""Host logic of the sampler rule "the first 25 % of the denoising steps use full attention" (Section 4.1)."""
import pytest

from paper_2506_23858_b200.layer import dense_step_schedule


def test_first_quarter_of_the_steps_is_dense():
    s = dense_step_schedule(50)
    assert s[:13] == [True] * 13 and s[13:] == [False] * 37          # ceil(12.5) = 13 of 50 steps
    assert dense_step_schedule(40) == [True] * 10 + [False] * 30


def test_schedule_edges():
    assert dense_step_schedule(0) == []
    assert dense_step_schedule(4, 0.0) == [False] * 4
    assert dense_step_schedule(4, 1.0) == [True] * 4
    assert dense_step_schedule(1) == [True]                           # ceil(0.25) = 1
    assert dense_step_schedule(8, 0.25) == [True, True] + [False] * 6
    with pytest.raises(ValueError):
        dense_step_schedule(4, 1.5)
    with pytest.raises(ValueError):
        dense_step_schedule(-1)


def test_schedule_is_a_prefix_and_monotone_in_the_fraction():
    for n in (1, 7, 50):
        prev = 0
        for f in (0.0, 0.1, 0.25, 0.5, 1.0):
            s = dense_step_schedule(n, f)
            k = sum(s)
            assert s == [True] * k + [False] * (n - k) and k >= prev
            prev = k
