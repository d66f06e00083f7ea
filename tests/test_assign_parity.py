"""Parity of dynamo_assign_bits (host code behind the C-ABI) with the Algorithm 1 oracle: memberships and
centers within 1e-9 (both sides are float64; they differ in the order of the arithmetic), iteration counts, hard
clusters and bits exact.  Host-only entry point: runs without a GPU."""
import numpy as np
import pytest

from oracle import assign as A
from paper_2503_21135_b200 import binding

TOL = 1e-9
ERR = binding.STATUS_NAMES.index


def _problem(seed, n, c, dim):
    rng = np.random.default_rng(seed)
    # significance with a few well-populated levels plus stragglers, like expert loads under a skewed router
    x = np.abs(rng.choice([0.1, 0.3, 0.6, 1.0], size=(n, dim)) + 0.05 * rng.standard_normal((n, dim)))
    u0 = rng.random((n, c)) + 0.05
    u0 /= u0.sum(axis=1, keepdims=True)
    return x, u0


@pytest.mark.parametrize("n,c,dim,m", [(8, 4, 1, 2.0), (64, 4, 1, 2.0), (64, 4, 1, 1.5), (66, 3, 2, 3.0), (5, 5, 1, 2.0),
                                        (200, 4, 3, 2.0)])
def test_parity_random_init(n, c, dim, m):
    x, u0 = _problem(n + c, n, c, dim)
    levels = [8, 6, 4, 3, 2][:c]
    got = binding.assign_bits(x, levels, c=c, m=m, eps=1e-10, max_iter=2000, u0=u0, overlap=0.02)
    V, U, it, _ = A.fuzzy_cmeans(x.tolist(), u0.tolist(), m=m, eps=1e-10, max_iter=2000)
    bits, hard = A.assign_bits(V, U, levels, overlap=0.02)
    assert got["iters"] == it
    assert np.max(np.abs(got["U"] - np.array(U))) <= TOL and np.max(np.abs(got["V"] - np.array(V))) <= TOL
    # a membership margin within TOL of the overlap threshold could legitimately flip: none here
    top2 = np.sort(np.array(U), axis=1)[:, -2:]
    assert np.all(np.abs((top2[:, 1] - top2[:, 0]) - 0.02) > 1e-6)
    assert got["bits"].tolist() == bits and got["cluster"].tolist() == hard


@pytest.mark.parametrize("c", [1, 2, 4])
def test_parity_token_share_init(c):
    rng = np.random.default_rng(5)
    share = rng.dirichlet(np.full(16, 0.7))
    x = share * 3.0 + 0.01 * rng.random(16)
    levels = [8, 4, 3, 2][:c]
    got = binding.assign_bits(x, levels, c=c, token_share=share, max_iter=1)
    U0 = A.initial_memberships(share.tolist(), c, 2.0)
    V, U, it, _ = A.fuzzy_cmeans(x[:, None].tolist(), U0, m=2.0, eps=1e-9, max_iter=1)
    assert np.max(np.abs(got["U"] - np.array(U))) <= TOL and np.max(np.abs(got["V"] - np.array(V))) <= TOL
    full = binding.assign_bits(x, levels, c=c, token_share=share)
    V, U, it, _ = A.fuzzy_cmeans(x[:, None].tolist(), U0, m=2.0, eps=1e-9, max_iter=1000)
    assert full["iters"] == it and np.max(np.abs(full["U"] - np.array(U))) <= TOL
    assert full["bits"].tolist() == A.assign_bits(V, U, levels)[0]
    # equal shares: flat start, every cluster gets the same center, the exact tie resolves to the lowest precision
    flat = binding.assign_bits(x, levels, c=c, token_share=np.full(16, 1 / 16))
    assert np.all(flat["U"] == 1.0 / c) and flat["bits"].tolist() == [levels[-1]] * 16


def test_points_on_centers_and_exact_values():
    x = np.array([1.0, 5.0, 5.0, 1.0, 9.0])
    u0 = np.array([[1, 0, 0], [0, 1, 0], [0, 1, 0], [1, 0, 0], [0, 0, 1]], float)
    got = binding.assign_bits(x, [8, 4, 2], c=3, u0=u0)
    assert got["iters"] == 1 and got["V"].ravel().tolist() == [1.0, 5.0, 9.0]
    assert np.array_equal(got["U"], u0) and got["bits"].tolist() == [2, 4, 4, 2, 8]
    # the hand-worked iteration of the oracle's pin, through the library
    got = binding.assign_bits([0.0, 1.0], [8, 2], c=2, u0=[[0.8, 0.2], [0.2, 0.8]], eps=0.0, max_iter=1)
    assert got["V"].ravel() == pytest.approx([1 / 17, 16 / 17], abs=1e-15)
    assert got["U"][0] == pytest.approx([256 / 257, 1 / 257], abs=1e-15)
    assert got["bits"].tolist() == [2, 8]


def test_expert_loads_to_bits_config_shapes():
    # 8 experts under a Zipf router (config 2/3 shape) and 64 fine-grained experts (config 4 shape)
    for n, seed in ((8, 0), (64, 1)):
        rng = np.random.default_rng(seed)
        share = np.sort(rng.zipf(1.6, n).astype(float))
        share /= share.sum()
        got = binding.assign_bits(share, [8, 4, 3, 2], token_share=share, overlap=0.1)
        U0 = A.initial_memberships(share.tolist(), 4, 2.0)
        V, U, it, _ = A.fuzzy_cmeans(share[:, None].tolist(), U0)
        assert got["bits"].tolist() == A.assign_bits(V, U, [8, 4, 3, 2], overlap=0.1)[0]
        assert np.all(np.diff(got["bits"]) >= 0)            # more load never means fewer bits
        assert got["bits"][-1] == 8 and got["bits"][0] == 2


def test_errors():
    x, u0 = _problem(0, 8, 4, 1)
    ok = dict(c=4, u0=u0)
    with pytest.raises(binding.DynamoError) as ei:
        binding.assign_bits(x, [8, 4, 3, 2], c=4)
    assert ei.value.status == ERR("ERR_NULL")
    for kw, code in ((dict(ok, m=1.0), "ERR_ARG"), (dict(ok, eps=-1.0), "ERR_ARG"), (dict(ok, overlap=-0.1), "ERR_ARG"),
                     (dict(ok, max_iter=0), "ERR_SHAPE"), (dict(c=4, u0=u0 * 1.01), "ERR_ARG"),
                     (dict(c=4, u0=np.where(np.arange(4) == 0, 1.0, 0.0) * np.ones((8, 1))), "ERR_ARG")):
        with pytest.raises(binding.DynamoError) as ei:
            binding.assign_bits(x, [8, 4, 3, 2], **kw)
        assert ei.value.status == ERR(code), kw
    with pytest.raises(binding.DynamoError) as ei:
        binding.assign_bits(x, [8, 5, 3, 2], **ok)
    assert ei.value.status == ERR("ERR_BITS")
    with pytest.raises(binding.DynamoError) as ei:
        binding.assign_bits(x[:3], [8, 4, 3, 2], c=4, u0=u0[:3])
    assert ei.value.status == ERR("ERR_SHAPE")
    bad = x.copy()
    bad[2, 0] = np.nan
    with pytest.raises(binding.DynamoError) as ei:
        binding.assign_bits(bad, [8, 4, 3, 2], **ok)
    assert ei.value.status == ERR("ERR_ARG")
