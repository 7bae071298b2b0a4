"""Pins of the speculative-sampling oracle (Sec. 3: accept by the ratio of target and drafter probabilities,
bonus token from the residual distribution) against what the rule guarantees and against library routines."""
import numpy as np
import pytest

import oracle


def softmax(x, T):
    z = (x.astype(np.float64) - x.max(-1, keepdims=True)) / T
    e = np.exp(z)
    return e / e.sum(-1, keepdims=True)


def one_step_inputs(rng, V, n, T, q_kind):
    """n independent sequences with one draft each (C = 2 rows), the same target / draft logits for all of them,
    draft tokens drawn from q, fresh uniforms: the first committed token of every sequence is one sample."""
    lp = rng.normal(size=(2, V)).astype(np.float32) * 1.5
    ld = (lp + rng.normal(size=(2, V)).astype(np.float32)) if q_kind == "noisy" else lp.copy()
    p0, q0 = softmax(lp[0], T), softmax(ld[0], T)
    logits = np.tile(lp, (n, 1)); dlog = np.tile(ld, (n, 1))
    x = rng.choice(V, size=n, p=q0)
    drafts = np.zeros((2 * n,), np.int32); drafts[1::2] = x
    return logits, dlog, drafts, p0, q0, x


@pytest.mark.parametrize("T", [0.3, 1.0])
@pytest.mark.parametrize("q_kind", ["noisy", "equal"])
def test_first_committed_token_follows_the_target_distribution(T, q_kind):
    """Losslessness: whatever q proposes, the token committed at the first position is distributed as p_0."""
    rng = np.random.default_rng(5)
    V, n = 7, 120_000
    logits, dlog, drafts, p0, q0, x = one_step_inputs(rng, V, n, T, q_kind)
    ql = np.full((n,), 2, np.int32); nm = np.zeros((n,), np.int32)
    ua = rng.random(2 * n, dtype=np.float32); ub = rng.random(n, dtype=np.float32)
    acc, bon, ratio = oracle.accept_stochastic(logits, dlog, drafts, ql, nm, T, ua, ub)
    first = np.where(acc >= 1, x, bon)                # accepted: the draft itself; rejected: the bonus token
    freq = np.bincount(first, minlength=V) / n
    sigma = np.sqrt(p0 * (1 - p0) / n)
    assert np.all(np.abs(freq - p0) < 4.5 * sigma + 1e-9), (freq, p0)
    if q_kind == "equal":                             # p == q: ratio 1, nothing is ever rejected
        assert (acc == 1).all() and np.allclose(ratio[0::2], 1.0)
    else:                                             # acceptance rate = sum_x min(p, q)
        assert abs((acc == 1).mean() - np.minimum(p0, q0).sum()) < 5e-3


def test_point_mass_drafter_accepts_with_probability_p_and_never_resamples_the_rejected_token():
    rng = np.random.default_rng(9)
    V, n, T = 6, 60_000, 0.6
    lp = rng.normal(size=(2, V)).astype(np.float32)
    p0 = softmax(lp[0], T)
    x = 2
    logits = np.tile(lp, (n, 1))
    drafts = np.zeros((2 * n,), np.int32); drafts[1::2] = x
    ql = np.full((n,), 2, np.int32); nm = np.zeros((n,), np.int32)
    ua = rng.random(2 * n, dtype=np.float32); ub = rng.random(n, dtype=np.float32)
    acc, bon, ratio = oracle.accept_stochastic(logits, None, drafts, ql, nm, T, ua, ub)
    assert np.allclose(ratio[0::2], p0[x])
    assert abs((acc == 1).mean() - p0[x]) < 4.5 * np.sqrt(p0[x] * (1 - p0[x]) / n)
    rej = acc == 0
    assert (bon[rej] != x).all()
    res = p0.copy(); res[x] = 0; res /= res.sum()     # residual of a point mass: p without x, renormalised
    freq = np.bincount(bon[rej], minlength=V) / rej.sum()
    assert np.all(np.abs(freq - res) < 4.5 * np.sqrt(res * (1 - res) / rej.sum()) + 1e-9)


def test_low_temperature_reduces_to_greedy_verification():
    """T -> 0 with a point-mass drafter: p is one-hot at the argmax, so a draft is accepted iff it is the argmax."""
    rng = np.random.default_rng(3)
    V, B = 500, 40
    C = rng.integers(1, 9, size=B)
    R = int(C.sum())
    logits = rng.normal(size=(R, V)).astype(np.float32)
    am = logits.argmax(-1)
    drafts = rng.integers(0, V, size=R).astype(np.int32)
    r0 = 0
    for c in C:
        for j in range(c - 1):
            if rng.random() < 0.8:
                drafts[r0 + j + 1] = am[r0 + j]
        r0 += c
    ql = C.astype(np.int32); nm = np.zeros((B,), np.int32)
    ua = rng.random(R, dtype=np.float32) * 0.999 + 0.0005; ub = rng.random(B, dtype=np.float32)
    acc, bon, _ = oracle.accept_stochastic(logits, None, drafts, ql, nm, 1e-3, ua, ub)
    r0 = 0
    for b, c in enumerate(C):                         # numpy replay with the library argmax
        a = 0
        while a < c - 1 and am[r0 + a] == drafts[r0 + a + 1]:
            a += 1
        assert acc[b] == a and bon[b] == am[r0 + a]
        r0 += c


def test_bonus_token_is_the_inverse_cdf_of_the_weights():
    """The draw is numpy's searchsorted on numpy's cumsum of the weights the oracle reports."""
    rng = np.random.default_rng(11)
    V, B, T = 300, 64, 0.8
    C = rng.integers(1, 6, size=B)
    R = int(C.sum())
    logits = rng.normal(size=(R, V)).astype(np.float32) * 2
    dlog = logits + rng.normal(size=(R, V)).astype(np.float32)
    drafts = rng.integers(0, V, size=R).astype(np.int32)
    ql = (C + 3).astype(np.int32); nm = np.full((B,), 3, np.int32)      # mask rows do not count
    ua = rng.random(R, dtype=np.float32); ub = rng.random(B, dtype=np.float32)
    ub[0], ub[1] = 0.0, np.float32(1.0 - 2 ** -24)
    acc, bon, ratio, w = oracle.accept_stochastic(logits, dlog, drafts, ql, nm, T, ua, ub, want_weights=True)
    r0 = 0
    for b, c in enumerate(C):
        cdf = np.cumsum(w[b])
        assert bon[b] == min(int(np.searchsorted(cdf, float(ub[b]) * cdf[-1], side="right")), V - 1)
        a = int(acc[b])
        assert 0 <= a <= c - 1
        p = softmax(logits[r0 + a], T)
        if a < c - 1:                                 # rejected at a: weights are the clipped difference
            qd = softmax(dlog[r0 + a], T)
            np.testing.assert_allclose(w[b], np.maximum(p - qd, 0), atol=1e-15)
            x = drafts[r0 + a + 1]
            assert ua[r0 + a] >= min(1.0, p[x] / qd[x])
        else:
            np.testing.assert_allclose(w[b], p, atol=1e-15)
        for j in range(a):                            # every earlier draft passed its test
            pj, qj = softmax(logits[r0 + j], T), softmax(dlog[r0 + j], T)
            x = drafts[r0 + j + 1]
            assert ua[r0 + j] < min(1.0, pj[x] / qj[x]) and abs(ratio[r0 + j] - pj[x] / qj[x]) < 1e-12
        r0 += c
    assert bon[0] == int(np.flatnonzero(w[0] > 0)[0])  # u = 0: the first token with any weight


def test_sequences_without_candidate_rows():
    acc, bon, _ = oracle.accept_stochastic(np.zeros((0, 5), np.float32), None, np.zeros((0,), np.int32), np.array([4], np.int32),
                                          np.array([4], np.int32), 1.0, np.zeros((0,), np.float32), np.zeros((1,), np.float32))
    assert acc[0] == -1 and bon[0] == -1


def test_draft_token_without_drafter_mass():
    """A draft the drafter itself gives probability 0 (Sec. 3's ratio p/q has no value there): the product form of
    the test, u q(x) < p(x), accepts it exactly when the target gives it mass, and rejects it when neither does."""
    V, T = 6, 1.0
    lp = np.zeros((3, 2, V), np.float32); ld = np.zeros((3, 2, V), np.float32)
    ld[:, 0, 2] = -np.inf                             # q_0(2) = 0 in every sequence
    lp[1, 0, 2] = -np.inf                             # sequence 1: p_0(2) = 0 as well
    lp[2, 0, :] = -np.inf; lp[2, 0, 2] = 0.0          # sequence 2: p_0 is a point mass on token 2
    drafts = np.zeros((6,), np.int32); drafts[1::2] = 2
    ql = np.full((3,), 2, np.int32); nm = np.zeros((3,), np.int32)
    for u in (0.0, 0.5, 0.999):
        ua = np.full((6,), u, np.float32); ub = np.full((3,), 0.3, np.float32)
        acc, bon, ratio = oracle.accept_stochastic(lp.reshape(6, V), ld.reshape(6, V), drafts, ql, nm, T, ua, ub)
        assert acc.tolist() == [1, 0, 1]
        assert bon[1] != 2                            # the residual of sequence 1 has no mass on the rejected token
