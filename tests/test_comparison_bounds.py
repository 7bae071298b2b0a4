"""What the two bounds of the long-context parity test can and cannot see (CPU only).  A kernel that loses one
128-token tile of a 32 800-token sequence, or gives one split partial a slightly wrong weight, changes every output
element by far less than the elementwise tolerance; the per-vector bound is what notices.  The mistakes are planted
in a plain float64 computation here, not in any kernel."""
import numpy as np
import pytest

from helpers import ATOL, RTOL, worst_vector_error


def _attention_rows(q, K, V, keep=None, weights=None):
    """softmax(q K^T / sqrt(d)) V for rows q [R, d] over keys K, V [N, d]; `keep`: boolean [N] of the keys that take
    part; `weights`: a factor per key applied to the unnormalised probabilities (a wrong split weight)."""
    s = (q @ K.T) / np.sqrt(q.shape[1])
    if keep is not None:
        s = np.where(keep[None, :], s, -np.inf)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    if weights is not None:
        p = p * weights[None, :]
    return (p / p.sum(axis=1, keepdims=True)) @ V


def _elementwise_ok(got, ref):
    return bool((np.abs(got - ref) <= ATOL + RTOL * np.abs(ref)).all())


@pytest.fixture(scope="module")
def long_rows():
    rng = np.random.default_rng(7)
    N, d, R = 32800, 128, 64
    bf = lambda a: a.astype(np.float32).view(np.uint32).__rshift__(16).__lshift__(16).view(np.float32).astype(np.float64)   # bf16 grid
    return bf(rng.standard_normal((R, d))), bf(rng.standard_normal((N, d))), bf(rng.standard_normal((N, d)))


def test_a_lost_tile_passes_the_elementwise_bound_and_fails_the_vector_bound(long_rows):
    q, K, V = long_rows
    ref = _attention_rows(q, K, V)
    keep = np.ones(K.shape[0], bool)
    keep[128 * 100:128 * 101] = False                        # one tile of 257 never reaches the softmax
    got = _attention_rows(q, K, V, keep=keep)
    assert _elementwise_ok(got, ref)                          # the benchmark spec's tolerance alone would let it through
    assert worst_vector_error(got, ref) > 2e-2                # ... the vector bound does not (about 6 % here)


def test_a_wrong_split_weight_is_noticed(long_rows):
    q, K, V = long_rows
    ref = _attention_rows(q, K, V)
    w = np.ones(K.shape[0])
    w[: K.shape[0] // 3] = 1.25                               # one of three partials merged with a weight 25 % too large
    got = _attention_rows(q, K, V, weights=w)
    assert _elementwise_ok(got, ref)
    assert worst_vector_error(got, ref) > 2e-2


def test_rounding_of_the_kernels_kind_stays_inside_both_bounds(long_rows):
    q, K, V = long_rows
    ref = _attention_rows(q, K, V)
    rng = np.random.default_rng(8)
    # probabilities rounded to bf16 before P V and the output rounded to bf16: relative 2^-9 each
    noisy = ref * (1 + rng.uniform(-2.0 ** -9, 2.0 ** -9, ref.shape)) + rng.uniform(-1, 1, ref.shape) * 2.0 ** -9 * np.abs(ref).mean()
    assert _elementwise_ok(noisy, ref)
    assert worst_vector_error(noisy, ref) < 1e-2
