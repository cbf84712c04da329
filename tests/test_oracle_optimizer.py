"""Pins for the oracle's layer-set suggestion engine (Section 4.1): random search with a Gaussian-process step
every beta-th proposal.  The Gaussian process is checked against scikit-learn's, the random sets against the
uniform law, the schedule against the paper's rule (o mod beta = 0), and the whole against a planted objective."""
import numpy as np
import pytest

from oracle import swift_oracle as so


def _planted_objective(planted, m, gamma=32):
    """matchness-like score: falls with every skipped block that is not planted; a multiple of 1 / gamma."""
    return lambda s: round((1.0 - len(set(s) - planted) / m) * gamma) / gamma


def test_random_sets_are_uniform_m_subsets():
    opt = so.LayerSetOptimizer(20, 7, seed=5)
    counts = np.zeros(20)
    n = 4000
    for _ in range(n):
        s = opt.random_set()
        assert len(s) == 7 and len(set(s)) == 7 and list(s) == sorted(s) and 0 <= s[0] and s[-1] < 20
        counts[list(s)] += 1
    # each block is in a uniform 7-subset with probability 7/20; binomial standard deviation sqrt(n p (1 - p)) = 30
    assert np.abs(counts - n * 7 / 20).max() < 4.5 * np.sqrt(n * 0.35 * 0.65)
    other = so.LayerSetOptimizer(20, 7, seed=6)
    assert [other.random_set() for _ in range(5)] != [so.LayerSetOptimizer(20, 7, seed=5).random_set() for _ in range(5)]


@pytest.mark.parametrize("ell", [1.0, 2.0, 4.0])
def test_gaussian_process_matches_scikit_learn(ell):
    from sklearn.gaussian_process import GaussianProcessRegressor
    from sklearn.gaussian_process.kernels import Matern
    opt = so.LayerSetOptimizer(12, 5, seed=1, noise=1e-2, ells=(ell,))
    f = _planted_objective({0, 2, 4, 6, 8}, 5)
    for _ in range(30):
        s = opt.random_set()
        opt.observe(s, f(s))
    model = opt.fit()
    assert model["ell"] == ell
    probe = [opt.random_set() for _ in range(40)]
    mean, std = opt.predict(model, probe)
    X = opt._indicator(opt.X)
    y = np.asarray(opt.y)
    # mean function: ridge regression of the standardised scores on the indicators, here by an augmented least-squares solve
    t = (y - y.mean()) / y.std()
    w = np.linalg.lstsq(np.vstack([X, np.sqrt(opt.ridge) * np.eye(12)]), np.concatenate([t, np.zeros(12)]), rcond=None)[0]
    assert np.allclose(model["w"], w, atol=1e-10)
    # the Gaussian process models the residuals (all 30 evaluations fit its window)
    gp = GaussianProcessRegressor(kernel=Matern(length_scale=ell, nu=2.5), alpha=1e-2, optimizer=None, normalize_y=False)
    gp.fit(X, t - X @ w)                                # Euclidean distance of indicator vectors = sqrt(Hamming distance)
    P = opt._indicator(probe)
    ref_mean, ref_std = gp.predict(P, return_std=True)
    assert np.allclose(mean, y.mean() + y.std() * (P @ w + ref_mean), atol=1e-9) and np.allclose(std, y.std() * ref_std, atol=1e-7)
    assert model["lml"] == pytest.approx(gp.log_marginal_likelihood_value_, abs=1e-8)


def test_gaussian_process_window_takes_the_most_recent_evaluations():
    opt = so.LayerSetOptimizer(12, 5, seed=4, gp_window=10, ells=(2.0,))
    f = _planted_objective({0, 2, 4, 6, 8}, 5)
    for _ in range(25):
        s = opt.random_set()
        opt.observe(s, f(s))
    model = opt.fit()
    assert model["X"].shape == (10, 12) and np.array_equal(model["X"], opt._indicator(opt.X[-10:]))
    y = np.asarray(opt.y)
    t = (y - y.mean()) / y.std()
    assert np.allclose(model["resid"], (t - opt._indicator(opt.X) @ model["w"])[-10:])


def test_length_scale_is_chosen_by_marginal_likelihood():
    opt = so.LayerSetOptimizer(12, 5, seed=2)
    f = _planted_objective({1, 3, 5, 7, 9}, 5)
    for _ in range(25):
        s = opt.random_set()
        opt.observe(s, f(s))
    chosen = opt.fit()
    each = []
    for ell in opt.ells:
        one = so.LayerSetOptimizer(12, 5, seed=2, ells=(ell,))
        one.X, one.y = opt.X, opt.y
        each.append(one.fit()["lml"])
    assert chosen["lml"] == max(each) and chosen["ell"] == opt.ells[int(np.argmax(each))]


def test_every_beta_th_step_is_bayesian_and_maximises_the_bound():
    opt = so.LayerSetOptimizer(16, 6, beta=4, seed=9, pool=50)
    f = _planted_objective({0, 1, 2, 3, 4, 5}, 6)
    kinds = []
    for step in range(1, 17):
        shadow = so.LayerSetOptimizer(16, 6, beta=0, seed=9)
        shadow.draws = opt.draws
        would_be_random = shadow.random_set()
        s = opt.suggest()
        assert opt.step == step and s not in opt.X or step % 4 != 0
        kinds.append(s != would_be_random)
        opt.observe(s, f(s))
    assert [k for i, k in enumerate(kinds, 1) if i % 4 != 0] == [False] * 12      # random search in between
    assert all(k for i, k in enumerate(kinds, 1) if i % 4 == 0)                   # o mod beta = 0: Bayesian
    pick, info = opt.bayesian_set()
    assert pick not in opt.X and info["ucb"] == pytest.approx(float(np.max(info["ucb_all"])))
    inc = opt.best_set()
    swaps = {tuple(sorted((set(inc) - {a}) | {b})) for a in inc for b in range(16) if b not in inc}
    assert swaps - set(opt.X) <= set(info["candidates"])                           # every one-swap neighbour is considered
    cheapest = tuple(sorted(sorted(range(16), key=lambda b: (-round(float(info["model"]["w"][b]), 6), b))[:6]))
    assert cheapest in set(info["candidates"]) | set(opt.X)                        # and the regression's own best guess


def test_finds_a_planted_set_that_random_search_misses():
    """40 blocks, 18 of them free to skip, score falling by 1/18 per other block skipped: with the Gaussian-process step
    every 25th proposal the search reaches 0.9 well within S = 1000 steps; random search alone does not."""
    planted = set(range(1, 37, 2))
    f = _planted_objective(planted, 18)
    bo = so.LayerSetOptimizer(40, 18, beta=25, seed=0)
    best_at = None
    for step in range(1, 1001):
        s = bo.suggest()
        bo.observe(s, f(s))
        if f(s) >= 0.9 and best_at is None:
            best_at = step
            break
    assert best_at is not None and best_at <= 300, best_at
    rs = so.LayerSetOptimizer(40, 18, beta=0, seed=0)
    assert max(f(rs.suggest()) for _ in range(1000)) < 0.9
