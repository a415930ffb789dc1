"""The speed-up model of Sec. III-B/III-C (Eq. 1) against the paper's worked numbers, and the round accountant against
Eq. 1 (an identity once alpha is taken as the accepted fraction the simulation actually saw)."""
import random

import pytest

from paper_2503_13565_b200 import specdec


def test_eq1_worked_examples_of_the_paper():
    # Sec. III-B: N = 4 gives (alpha + 0.25) / (1/S + 0.25); a 4x faster draft at 85 % acceptance: 2.2x
    assert specdec.eq1_speedup(0.85, 4, 4.0) == pytest.approx((0.85 + 0.25) / (0.25 + 0.25))
    assert specdec.eq1_speedup(0.85, 4, 4.0) == pytest.approx(2.2)
    # both forms of Eq. 1 agree: (G + 1) / (1 + N / S)
    for g, n, s in [(3, 4, 4.0), (2, 8, 20.0), (0, 4, 100.0), (8, 8, 3.76)]:
        assert specdec.eq1_speedup(g / n, n, s) == pytest.approx((g + 1) / (1 + n / s))
    # a draft that is never right still yields the target's own token per round: slower than no draft at all
    assert specdec.eq1_speedup(0.0, 4, 4.0) == pytest.approx(0.5)


def test_two_level_example_of_the_paper():
    """Sec. III-C: BF16 target, 4-bit intermediate (4x faster), tiny draft (100x faster); 80-85 % and 40-45 % acceptance
    give 3-3.5x, where either draft alone gives 2-2.5x."""
    for a1, a2 in [(0.80, 0.40), (0.85, 0.45), (0.825, 0.425)]:
        two = specdec.multilevel_speedup([1.0, 1 / 4, 1 / 100], [4, 4], [a1, a2])
        assert 2.9 <= two <= 3.5, two
        one_q = specdec.multilevel_speedup([1.0, 1 / 4], [4], [a1])
        one_t = specdec.multilevel_speedup([1.0, 1 / 100], [4], [a2])
        assert 2.0 <= one_q <= 2.5 and one_t < two and one_q < two
    # one level reduces to Eq. 1
    assert specdec.multilevel_speedup([1.0, 0.25], [4], [0.85]) == pytest.approx(2.2)


@pytest.mark.parametrize("p,n,s", [(0.9, 4, 4.0), (0.7, 8, 3.76), (0.45, 4, 100.0)])
def test_accountant_equals_eq1_at_the_observed_acceptance(p, n, s):
    rng = random.Random(7)
    tally = specdec.simulate(2, [n], lambda lvl, k: specdec.leading_successes(rng, p, k), tokens=20000)
    rounds = tally.steps[0]
    assert tally.steps[1] == rounds * n and tally.proposed[0] == rounds * n
    alpha = tally.accepted[0] / tally.proposed[0]
    produced = tally.accepted[0] + rounds
    assert produced >= 20000
    t = tally.time([1.0, 1.0 / s])
    assert produced / t == pytest.approx(specdec.eq1_speedup(alpha, n, s), rel=1e-12)
    # and alpha itself is near its expectation sum_{i=1..N} p^i / N
    assert alpha == pytest.approx(sum(p ** i for i in range(1, n + 1)) / n, abs=0.02)


def test_two_level_accountant_close_to_the_nested_formula():
    rng = random.Random(11)
    n, p = [4, 4], [0.9, 0.6]
    tally = specdec.simulate(3, n, lambda lvl, k: specdec.leading_successes(rng, p[lvl], k), tokens=200000)
    alpha = [tally.accepted[i] / tally.proposed[i] for i in range(2)]
    produced = tally.accepted[0] + tally.steps[0]
    times = [1.0, 0.25, 0.01]
    got = produced / tally.time(times)
    # The nested formula charges the intermediate level its average time per token.  The rounds below ask it for
    # exactly N tokens, and its last round may yield more than were asked for (G + 1 up to N + 1); the surplus is
    # thrown away here and counted as useful by the formula.  So the formula is an upper bound, about 10 % away.
    model = specdec.multilevel_speedup(times, n, alpha)
    assert 0.85 * model <= got <= model


def test_on_step_sees_every_pass():
    seen = []
    specdec.simulate(2, [3], lambda lvl, k: 1, tokens=10, on_step=lambda lvl, rows: seen.append((lvl, rows)))
    assert seen[:4] == [(1, 1), (1, 1), (1, 1), (0, 4)] and len(seen) == 5 * 4


class _TableModel:
    """A deterministic stand-in: the next token is a fixed function of (token, position); `wrong_every` makes the model
    disagree with the reference function at some positions, as a draft would."""

    def __init__(self, v, salt, wrong_every=0):
        self.v, self.salt, self.wrong_every = v, salt, wrong_every
        self.passes = 0

    def choice(self, tok, pos):
        t = (tok * 31 + pos * 17 + 7) % self.v
        if self.wrong_every and (tok + pos + self.salt) % self.wrong_every == 0:
            t = (t + 1) % self.v
        return t

    def next(self, cur, pos):
        self.passes += 1
        return self.choice(cur, pos)

    def verify(self, cur, pos, proposals):
        self.passes += 1
        rows = [cur] + list(proposals)
        mine = [self.choice(t, pos + j) for j, t in enumerate(rows)]
        g = 0
        while g < len(proposals) and proposals[g] == mine[g]:
            g += 1
        return g, mine[g]


@pytest.mark.parametrize("levels,n", [(1, []), (2, [4]), (2, [1]), (3, [4, 3]), (3, [8, 2])])
def test_decode_reproduces_the_targets_own_greedy_decoding(levels, n):
    target = _TableModel(97, 0)
    models = [target] + [_TableModel(97, 3 + i, wrong_every=3 + 2 * i) for i in range(levels - 1)]
    out, tally = specdec.decode(models, n, first_token=5, tokens=300)
    want, cur = [], 5
    for pos in range(len(out)):
        cur = target.choice(cur, pos)
        want.append(cur)
    assert out == want and len(out) >= 300
    assert tally.steps == [m.passes for m in models]
    for i in range(levels - 1):
        assert tally.proposed[i] == tally.steps[i] * n[i] and 0 < tally.accepted[i] < tally.proposed[i]
    if levels == 2:   # Eq. 1 at the observed acceptance, with a draft step S times cheaper than a target step
        s = 4.0
        alpha = tally.accepted[0] / tally.proposed[0]
        produced = tally.accepted[0] + tally.steps[0]
        assert produced == len(out)
        assert produced / tally.time([1.0, 1.0 / s]) == pytest.approx(specdec.eq1_speedup(alpha, n[0], s), rel=1e-12)
