"""Pins of the oracle's random numbers and acceptance rule (Eq. 5, Algorithm 1's
acceptance part): published known-answer vectors, brute force, and the exact
output law of speculative sampling."""
import numpy as np
import pytest

from oracle import pacer_oracle as orc


def _kat_vectors():
    """tests/golden/philox4x32_10_kat.txt: counter(4) key(2) expected(4), hex."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    out = []
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 10:
            v = [int(t, 16) for t in line]
            out.append((v[:4], v[4:6], v[6:]))
    return out


def test_philox_known_answers():
    vec = _kat_vectors()
    assert len(vec) == 3
    for ctr, key, exp in vec:
        assert list(orc.philox(ctr, key)) == exp


def test_uniform_is_open_interval_and_flat():
    u = np.array([orc.uniform(42, v, 3, 0, 1) for v in range(40000)])
    assert u.min() > 0.0 and u.max() < 1.0
    hist, _ = np.histogram(u, bins=20, range=(0, 1))
    chi2 = ((hist - 2000.0) ** 2 / 2000.0).sum()
    assert chi2 < 43.8          # chi-square 19 dof, p = 0.001
    # four consecutive vocabulary indices share one Philox block: words 0..3
    blk = orc.philox([5, 3, 0, 1], [42, 0])
    for j in range(4):
        assert orc.uniform(42, 20 + j, 3, 0, 1) == ((int(blk[j]) >> 8) + 0.5) / 2 ** 24


def test_greedy_rule_is_longest_matching_prefix():
    rng = np.random.default_rng(0)
    V = 9
    for trial in range(200):
        gamma = int(rng.integers(1, 7))
        plog = rng.normal(size=(gamma + 1, V))
        top = plog.argmax(1)
        y = top[:gamma].copy()
        cut = int(rng.integers(0, gamma + 1))        # first mismatch at `cut` (none if == gamma)
        if cut < gamma:
            y[cut] = (y[cut] + 1 + rng.integers(0, V - 1)) % V
            y[cut + 1:] = rng.integers(0, V, size=gamma - cut - 1)   # later matches must not count
        n, nxt, _, _ = orc.accept_rule(plog, np.zeros((gamma, V)), y, mode=0)
        assert n == cut
        assert nxt == top[cut]


def test_greedy_tie_takes_lowest_index():
    plog = np.zeros((2, 5))
    plog[0, [1, 3]] = 2.0
    plog[1, [2, 4]] = 1.0
    n, nxt, mt, _ = orc.accept_rule(plog, np.zeros((1, 5)), [1], mode=0)
    assert (n, nxt) == (1, 2) and mt == 0.0
    n, nxt, _, _ = orc.accept_rule(plog, np.zeros((1, 5)), [3], mode=0)
    assert (n, nxt) == (0, 1)


def _softmax(v):
    e = np.exp(v - v.max())
    return e / e.sum()


@pytest.mark.parametrize("V", [8, 16])
def test_speculative_sampling_reproduces_target_distribution(V):
    """Leviathan et al.'s identity (cited by Section 2.2): if y ~ q, it is kept
    with probability min(1, p/q) and otherwise replaced by a draw from
    norm(max(0, p - q)), then the result is distributed as p.  Checked on the
    oracle's rule by chi-square over 30000 seeds; y is drawn here with numpy."""
    rng = np.random.default_rng(V)
    plog = rng.normal(size=(2, V)) * 1.5
    qlog = rng.normal(size=(1, V)) * 1.5
    p, q = _softmax(plog[0]), _softmax(qlog[0])
    N = 30000
    ys = rng.choice(V, size=N, p=q)
    out = np.zeros(V)
    n_acc = 0
    for s in range(N):
        n, nxt, _, _ = orc.accept_rule(plog, qlog, [ys[s]], mode=1, seed=1000 + s, pos_first=5)
        n_acc += n
        out[ys[s] if n == 1 else nxt] += 1
    chi2 = ((out - N * p) ** 2 / (N * p)).sum()
    crit = {8: 24.3, 16: 37.7}[V]                 # p = 0.001 at V-1 dof
    assert chi2 < crit, (chi2, out / N, p)
    beta = np.minimum(p, q).sum()                  # exact acceptance probability
    assert abs(n_acc / N - beta) < 4 * np.sqrt(beta * (1 - beta) / N)


def test_bonus_token_is_a_draw_from_the_last_row():
    """All drafts accepted (p == q makes alpha = 1): the next token ~ p_{gamma+1}."""
    rng = np.random.default_rng(3)
    V, N = 8, 20000
    plog = rng.normal(size=(2, V))
    qlog = plog[:1].copy()
    p_last = _softmax(plog[1])
    out = np.zeros(V)
    for s in range(N):
        n, nxt, _, _ = orc.accept_rule(plog, qlog, [s % V], mode=1, seed=s, pos_first=2)
        assert n == 1
        out[nxt] += 1
    assert ((out - N * p_last) ** 2 / (N * p_last)).sum() < 24.3


def test_residual_never_returns_a_token_with_p_below_q():
    rng = np.random.default_rng(4)
    V = 12
    plog, qlog = rng.normal(size=(2, V)) * 2, rng.normal(size=(1, V)) * 2
    p, q = _softmax(plog[0]), _softmax(qlog[0])
    y = int(np.argmax(q - p))                     # the most over-proposed token
    for s in range(3000):
        n, nxt, _, _ = orc.accept_rule(plog, qlog, [y], mode=1, seed=s)
        if n == 0:
            assert p[nxt] > q[nxt]
