"""Pins for the CPU oracle's greedy verification and KV commit."""
import numpy as np
import torch

import oracle
from paper_2605_20022_b200 import workload as wl


def test_argmax_hits_planted_target_and_numpy_argmax():
    step = wl.workload(0)
    logits, drafts, target = wl.make_logits(step)
    acc, bon, am = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    np.testing.assert_array_equal(am, target.numpy())
    np.testing.assert_array_equal(am, np.argmax(logits.numpy(), axis=1))


def replay(am, drafts, cand):
    """Independent restatement with numpy: longest run of drafts equal to the target
    token of the row before them (Sec. 3), bonus = target token where the run stops."""
    acc, bon, r0 = [], [], 0
    for C in cand:
        if C == 0:
            acc.append(-1); bon.append(-1); continue
        ok = am[r0:r0 + C - 1] == drafts[r0 + 1:r0 + C]
        a = int(np.argmin(np.append(ok, False)))      # index of the first mismatch
        acc.append(a); bon.append(int(am[r0 + a])); r0 += C
    return np.array(acc, np.int32), np.array(bon, np.int32)


def test_accept_matches_numpy_replay_on_ragged_batch():
    shape = wl.Shape(4, 2, 32, 257)
    step = wl.make_step("acc", shape, [5] * 7, [17, 1, 9, 4, 16, 3, 16], [0, 0, 4, 4, 0, 2, 16], seed=77, p_match=0.8)
    logits, drafts, target = wl.make_logits(step)
    acc, bon, am = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    ra, rb = replay(np.argmax(logits.numpy(), axis=1), drafts.numpy(), step.cand_rows.tolist())
    np.testing.assert_array_equal(acc, ra)
    np.testing.assert_array_equal(bon, rb)
    k = step.cand_rows.numpy() - 1
    assert ((acc <= k) & ((acc >= 0) | (k < 0))).all()
    assert acc[6] == -1 and bon[6] == -1              # a sequence with no candidate rows


def test_all_match_and_first_row_mismatch():
    shape = wl.Shape(4, 2, 32, 500)
    step = wl.make_step("all", shape, [5, 5], [9, 6], [0, 2], seed=78, p_match=1.0)
    logits, drafts, target = wl.make_logits(step)
    acc, bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    np.testing.assert_array_equal(acc, [8, 3])                      # accepted_len = k
    np.testing.assert_array_equal(bon, [int(target[8]), int(target[12])])  # argmax at the last verified row
    drafts2 = drafts.clone()
    drafts2[1] = (int(target[0]) + 1) % 500           # first draft of sequence 0 wrong
    acc, bon, _ = oracle.accept(logits, drafts2, step.q_lens, step.n_mask)
    assert acc[0] == 0 and bon[0] == int(target[0]) and acc[1] == 3
    drafts3 = drafts.clone()
    drafts3[5] = (int(target[4]) + 3) % 500           # a mismatch in the middle hides later matches
    acc, bon, _ = oracle.accept(logits, drafts3, step.q_lens, step.n_mask)
    assert acc[0] == 4 and bon[0] == int(target[4])


def test_ties_take_lowest_index_and_infinities_compare():
    V = 37
    logits = np.zeros((3, V), np.float32)
    logits[0, [5, 9, 30]] = 2.0                       # three-way tie
    logits[1, :] = -np.inf; logits[1, 12] = -1e30      # everything else -inf
    logits[2, 3] = np.inf; logits[2, 20] = np.inf      # +inf tie
    acc, bon, am = oracle.accept(logits, np.array([0, 5, 12], np.int32), np.array([3]), np.array([0]))
    np.testing.assert_array_equal(am, [5, 12, 3])
    assert acc[0] == 2 and bon[0] == 3
    flat = np.zeros((1, V), np.float32)                # all equal -> index 0
    _, bon, am = oracle.accept(flat, np.array([0], np.int32), np.array([1]), np.array([0]))
    assert am[0] == 0 and bon[0] == 0


def test_accept_length_statistics_follow_independence_closed_form():
    """Eq. 5's independence model: with iid match probability p, P(len >= i) = p^i."""
    B, k, p, V = 20000, 8, 0.8, 16
    shape = wl.Shape(4, 2, 32, V)
    step = wl.make_step("stat", shape, [0] * B, [k + 1] * B, [0] * B, seed=79, p_match=p, spare=0)
    logits, drafts, _ = wl.make_logits(step)
    acc, _, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    for i in range(1, k + 1):
        est, exact = float((acc >= i).mean()), p ** i
        assert abs(est - exact) < 4.5 * np.sqrt(exact * (1 - exact) / B), (i, est, exact)
    mean_exact = p * (1 - p ** k) / (1 - p)
    assert abs(acc.mean() - mean_exact) < 0.06


def pages_by_set_logic(step, acc, P=16):
    """Token-level restatement: a page stays iff it holds a token that is kept."""
    pt, pl = step.page_table.numpy().copy(), step.prefix_lens.numpy().copy()
    freed = []
    for b in range(step.batch):
        if acc[b] < 0:
            continue
        kv_len = int(pl[b] + step.q_lens[b])
        new_len = int(pl[b] + acc[b] + 1)
        held = {j // P for j in range(kv_len)}
        kept = {j // P for j in range(new_len)}
        for pg in sorted(held - kept):
            freed.append(int(pt[b, pg])); pt[b, pg] = -1
        pl[b] = new_len
    return pt, pl, np.array(freed, np.int32)


def test_commit_matches_token_level_set_logic_and_invariants():
    shape = wl.Shape(4, 2, 32, 100)
    g = torch.Generator().manual_seed(5)
    B = 40
    n = torch.randint(0, 200, (B,), generator=g).tolist()
    C = torch.randint(0, 17, (B,), generator=g)
    M = torch.randint(0, 2, (B,), generator=g) * 16
    step = wl.make_step("commit", shape, n, (C + M).tolist(), M.tolist(), seed=80, extra_table_cols=3)
    acc = np.array([int(torch.randint(0, int(c), (1,), generator=g)) if c > 0 else -1 for c in C], np.int32)
    pt, pl, freed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, acc)
    ept, epl, efreed = pages_by_set_logic(step, acc)
    np.testing.assert_array_equal(pt, ept)
    np.testing.assert_array_equal(pl, epl)
    np.testing.assert_array_equal(freed, efreed)
    old = step.page_table.numpy()
    for b in range(B):
        if acc[b] < 0:
            np.testing.assert_array_equal(pt[b], old[b]); assert pl[b] == n[b]; continue
        assert pl[b] == n[b] + acc[b] + 1 <= n[b] + int(C[b])          # L_acc = r_acc + 1, never past the candidates
        keep = -(-int(pl[b]) // 16)
        assert (pt[b, keep:] == -1).all() and (pt[b, :keep] == old[b, :keep]).all() and (pt[b, :keep] >= 0).all()
    before = set(old[old >= 0].tolist())
    after = set(pt[pt >= 0].tolist())
    assert after.isdisjoint(freed.tolist()) and after | set(freed.tolist()) == before
    assert len(set(freed.tolist())) == len(freed)


def test_lossless_toy_decode_loop():
    """Tokens committed by draft -> verify -> accept -> commit equal plain greedy decoding
    of the same toy target (a fixed logits table indexed by the previous token)."""
    V, steps, k = 50, 60, 5
    rng = np.random.default_rng(3)
    table = rng.standard_normal((V, V)).astype(np.float32)
    nxt = np.argmax(table, axis=1)
    greedy = [7]
    for _ in range(400):
        greedy.append(int(nxt[greedy[-1]]))
    # speculative loop: sequence = committed tokens; `bonus` is committed-but-not-yet-fed
    committed, bonus = [], 7
    P = 16
    prefix_len = 0
    table_pages = np.full((1, 64), -1, np.int32)
    free = list(range(63, -1, -1))
    for _ in range(steps):
        drafts, prev = [], bonus
        for _ in range(k):                            # a drafter that is right 70 % of the time
            t = int(nxt[prev]) if rng.random() < 0.7 else int(rng.integers(V))
            drafts.append(t); prev = t
        fed = [bonus] + drafts
        need = -(-(prefix_len + len(fed)) // P)       # append-then-attend: allocate pages for the block
        for pg in range(need):
            if table_pages[0, pg] < 0:
                table_pages[0, pg] = free.pop()
        logits = table[fed]                            # target logits at every candidate row
        acc, bon, _ = oracle.accept(logits, np.array(fed, np.int32), np.array([len(fed)]), np.array([0]))
        pt, pl, freed = oracle.commit(table_pages, np.array([prefix_len], np.int32), np.array([len(fed)]), acc)
        committed += fed[:int(acc[0]) + 1]
        assert pl[0] == len(committed)
        free += freed.tolist()[::-1]
        table_pages, prefix_len, bonus = pt, int(pl[0]), int(bon[0])
    assert committed == greedy[:len(committed)] and bonus == greedy[len(committed)]
    assert len(committed) > steps                      # some drafts were accepted
    assert sorted(free + table_pages[table_pages >= 0].tolist()) == list(range(64))
