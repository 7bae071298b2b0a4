"""Pins for the oracle's draft-side tail: calibrated argmax and confidence (Eq. 4), cumulative confidence
and verify length (Eq. 5)."""
import numpy as np
import torch

import oracle


def make(B=5, V=300, seed=0, M=(12, 0, 8, 6, 16), nb=(3, 1, 2, 0, 4)):
    g = torch.Generator().manual_seed(seed)
    Rm = sum(M)
    logits = torch.randn((Rm, V), generator=g) * 3
    bias = torch.randn((Rm, V), generator=g)
    return logits, bias, np.array(M, np.int32), np.array(nb, np.int32)


def test_tokens_and_confidence_against_library_softmax():
    logits, bias, M, nb = make()
    tok, pr, cum, keep, gap = oracle.draft_select(logits, bias, M, nb, 0.3, max_blocks=4, want_gap=True)
    x = logits.double() + bias.double()                          # Eq. 4's sum, exact in float64 for float32 inputs
    np.testing.assert_array_equal(tok, x.argmax(dim=1).numpy())
    ref = torch.softmax(x, dim=1)[torch.arange(x.shape[0]), torch.from_numpy(tok).long()]
    np.testing.assert_allclose(pr, ref.numpy(), rtol=1e-12)
    top2 = torch.topk(x, 2, dim=1).values
    np.testing.assert_allclose(gap, (top2[:, 0] - top2[:, 1]).numpy(), rtol=0, atol=0)
    # without a bias the logits themselves decide
    tok0, pr0, _, _ = oracle.draft_select(logits, None, M, nb, 0.3, max_blocks=4)
    np.testing.assert_array_equal(tok0, logits.argmax(dim=1).numpy())
    assert (tok0 != tok).any()                                   # the calibration changes some drafts


def test_first_token_as_the_calibrated_argmax():
    """Index 0 wins only because of its bias (and, in the second row, loses only because of it): the first element
    of a row takes part in Eq. 4's sum like every other."""
    V = 50
    g = torch.Generator().manual_seed(5)
    logits = torch.randn((2, V), generator=g); bias = torch.zeros((2, V))
    logits[0, 0] = logits[0].max() - 1.0; bias[0, 0] = 4.0       # wins by its bias
    logits[1, 0] = logits[1].max() + 1.0; bias[1, 0] = -6.0      # would win without it
    tok, pr, _, _ = oracle.draft_select(logits, bias, np.array([2], np.int32), None, 0.5, max_blocks=1)
    x = logits.double() + bias.double()
    assert tok[0] == 0 and tok[1] == int(x[1].argmax()) != 0
    ref = torch.softmax(x, dim=1)[torch.arange(2), torch.from_numpy(tok).long()]
    np.testing.assert_allclose(pr, ref.numpy(), rtol=1e-12)


def test_sum_is_not_rounded_to_float32():
    """Two calibrated logits that a float32 sum makes equal (lower index would win) but whose exact sums differ."""
    V = 8
    logits = np.zeros((1, V), np.float32); bias = np.zeros((1, V), np.float32)
    logits[0, 2] = 1.0; bias[0, 2] = 2.0 ** -26                 # 1 + 2^-26 rounds to 1 in float32
    logits[0, 5] = 1.0; bias[0, 5] = 2.0 ** -25                 # so does 1 + 2^-25, the larger exact sum
    assert np.float32(logits[0, 2] + bias[0, 2]) == np.float32(logits[0, 5] + bias[0, 5])
    tok, pr, cum, keep, gap = oracle.draft_select(logits, bias, np.array([1], np.int32), None, 0.5, max_blocks=1, want_gap=True)
    assert tok[0] == 5
    assert 0 < gap[0] < 1e-7


def test_cumulative_confidence_and_keep_len_against_numpy():
    logits, bias, M, nb = make(seed=1)
    for thr in (0.9, 0.2, 1e-3, 0.0, 1.5):
        tok, pr, cum, keep = oracle.draft_select(logits, bias, M, nb, thr, max_blocks=4)
        r0 = 0
        for b in range(len(M)):
            n_b = max(int(nb[b]), 1)
            kb = int(M[b]) // n_b if M[b] else 0
            for g in range(4):
                if M[b] == 0 or g >= n_b:
                    assert keep[b, g] == 0
                    continue
                p = pr[r0 + g * kb:r0 + (g + 1) * kb]
                c = np.cumprod(p)
                np.testing.assert_allclose(cum[r0 + g * kb:r0 + (g + 1) * kb], c, rtol=1e-13)
                ok = c >= thr
                assert keep[b, g] == (int(np.argmin(ok)) if not ok.all() else kb)      # leading run only
            r0 += int(M[b])
        if thr == 0.0:
            assert all(keep[b, g] == (M[b] // max(nb[b], 1)) for b in range(len(M)) for g in range(max(nb[b], 1)) if M[b])
        if thr == 1.5:
            assert (keep == 0).all()


def test_constant_confidence_closed_form():
    """Every position equally confident with probability p: keep_len = floor(log(thr) / log(p)), capped by the block."""
    V, kb = 64, 10
    for peak in (1.0, 3.0, 5.0):
        logits = torch.zeros((kb, V)); logits[:, 7] = peak
        p = np.exp(peak) / (np.exp(peak) + V - 1)
        for thr in (0.5, 0.1, 0.01):
            tok, pr, cum, keep = oracle.draft_select(logits, None, np.array([kb], np.int32), None, thr, max_blocks=1)
            np.testing.assert_allclose(pr, p, rtol=1e-12)
            expect = min(kb, int(np.floor(np.log(thr) / np.log(p) + 1e-12)))
            assert (tok == 7).all() and keep[0, 0] == expect


def test_cumulative_confidence_is_the_independence_estimate_of_eq5():
    """Eq. 5: if each drafted token is accepted independently with probability p_i, the probability that the
    accepted length reaches i is the cumulative product the oracle reports."""
    logits, bias, M, nb = make(B=1, V=40, seed=3, M=(8,), nb=(1,))
    logits = logits * 0.5 + 2.5 * torch.nn.functional.one_hot(torch.arange(8) * 3, 40)   # confident but not certain drafts
    tok, pr, cum, keep = oracle.draft_select(logits, None, M, nb, 0.05, max_blocks=1)
    rng = np.random.default_rng(0)
    trials = 200000
    acc = rng.random((trials, 8)) < pr[None, :]
    run = np.cumprod(acc, axis=1).sum(axis=1)                      # accepted length of each trial
    for i in range(1, 9):
        est = (run >= i).mean()
        assert abs(est - cum[i - 1]) < 4.5 * np.sqrt(cum[i - 1] * (1 - cum[i - 1]) / trials) + 1e-4
