"""Pins for the oracle's greedy verification step (CPU only).

Sec. III-A: after the target's forward pass, every drafted token after the
first mismatch is dropped; Sec. III-B: with G accepted the round yields G+1
tokens, the extra one being the target's own.  The oracle is compared with a
literal Python restatement on exhaustively enumerated tiny cases and with
planted cases.
"""
import itertools

import numpy as np

import oracle


def literal_accept(logit_rows, draft):
    """logit_rows: list of R lists; draft: list of T ints."""
    ver = []
    for row in logit_rows:
        best, idx = None, 0
        for v, x in enumerate(row):
            if x != x:  # NaN
                continue
            if x == float("-inf"):
                continue
            if best is None or x > best:
                best, idx = x, v
        ver.append(idx)
    g = len(draft)
    for i, d in enumerate(draft):
        if d != ver[i]:
            g = i
            break
    nxt = ver[g] if g < len(ver) else -1
    return g, nxt, ver


def test_exhaustive_tiny():
    t, v = 2, 3
    vals = [-1.0, 0.0, 1.0]
    for r in (t, t + 1):
        rows = list(itertools.product(vals, repeat=v))            # 27 possible rows
        all_logits = list(itertools.product(range(len(rows)), repeat=r))
        drafts = list(itertools.product(range(v), repeat=t))
        lg = np.array([[rows[i] for i in combo] for combo in all_logits], np.float32)  # [27^r, r, v]
        for d in drafts:
            dd = np.tile(np.array(d, np.int32), (lg.shape[0], 1))
            g, nxt = oracle.greedy_accept(lg, dd)
            for b in range(0, lg.shape[0], 7 if r == 3 else 1):
                wg, wn, _ = literal_accept(lg[b].tolist(), list(d))
                assert (g[b], nxt[b]) == (wg, wn), (lg[b], d)


def test_later_agreement_does_not_count():
    ver = np.array([[5, 6, 7, 8, 9]], np.int32)
    draft = np.array([[5, 6, 0, 8]], np.int32)
    g, nxt = oracle.greedy_accept_tokens(draft, ver)
    assert (g[0], nxt[0]) == (2, 7)


def test_all_accepted_with_and_without_bonus_row():
    draft = np.array([[1, 2, 3]], np.int32)
    g, nxt = oracle.greedy_accept_tokens(draft, np.array([[1, 2, 3, 4]], np.int32))
    assert (g[0], nxt[0]) == (3, 4)          # G + 1 tokens produced
    g, nxt = oracle.greedy_accept_tokens(draft, np.array([[1, 2, 3]], np.int32))
    assert (g[0], nxt[0]) == (3, -1)
    g, nxt = oracle.greedy_accept_tokens(draft, np.array([[9, 2, 3]], np.int32))
    assert (g[0], nxt[0]) == (0, 9)


def test_argmax_ties_nan_inf():
    lg = np.zeros((6, 8), np.float32)
    lg[0, [2, 5]] = 3.0                       # tie: lowest index
    lg[1, :] = np.nan                         # nothing comparable: 0
    lg[2, :] = np.nan
    lg[2, 6] = -5.0                           # the only number wins
    lg[3, :] = -np.inf                        # nothing above -inf: 0
    lg[4, 3] = np.inf
    lg[4, 1] = np.nan
    lg[5, 7] = 1e-30
    assert list(oracle.argmax(lg)) == [2, 0, 6, 0, 3, 7]


def test_bf16_logits_compare_as_their_values():
    # BF16 bit patterns: negative numbers have larger unsigned patterns; the compare must be by value
    vals = np.array([[-2.0, -1.0, 0.5, 0.25, -0.0, 0.0]], np.float32)
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)
    assert oracle.argmax(bits)[0] == 2
    vals = np.array([[-2.0, -1.0, -0.5, -3.0]], np.float32)
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)
    assert oracle.argmax(bits)[0] == 2
    # +0 and -0 are equal: the lower index wins
    bits = np.array([[0x8000, 0x0000, 0x8000]], np.uint16)
    assert oracle.argmax(bits)[0] == 0


def test_random_against_literal_and_numpy():
    rng = np.random.default_rng(20)
    b, t, r, v = 40, 6, 7, 50
    lg = rng.standard_normal((b, r, v)).astype(np.float32)
    lg[rng.random((b, r, v)) < 0.05] = 1.5      # many exact ties
    ver = oracle.argmax(lg)
    assert np.array_equal(ver, np.argmax(lg, axis=-1).astype(np.int32))  # numpy: first maximum
    draft = ver[:, :t].copy()
    p = rng.integers(0, t + 1, b)
    for i in range(b):
        if p[i] < t:
            draft[i, p[i]] = (draft[i, p[i]] + 1 + rng.integers(0, v - 1)) % v
            for j in range(p[i] + 1, t):
                if rng.random() < 0.5:
                    draft[i, j] = rng.integers(0, v)
    g, nxt = oracle.greedy_accept(lg, draft)
    assert np.array_equal(g, p.astype(np.int32))
    for i in range(b):
        wg, wn, _ = literal_accept(lg[i].tolist(), draft[i].tolist())
        assert (g[i], nxt[i]) == (wg, wn)
