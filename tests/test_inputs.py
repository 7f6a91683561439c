"""The shared input generators: prime-chain rule and draw distributions."""
import numpy as np

from paper_2609_12378_b200 import inputs


def test_prime_chain_rule():
    for log_n, nq, npp in ((16, 24, 8), (13, 6, 1)):
        q, p = inputs.prime_chain(log_n, nq, npp)
        allp = [int(x) for x in p] + [int(x) for x in q]
        assert allp == sorted(allp, reverse=True) and len(set(allp)) == len(allp)
        for r in allp:
            assert (1 << 49) < r < (1 << 50) and r % (2 << log_n) == 1 and inputs.is_prime(r)
        # none skipped: every 1 mod 2N value between consecutive chain entries is composite
        m = 2 << log_n
        for hi, lo in zip(allp[:-1], allp[1:]):
            assert not any(inputs.is_prime(x) for x in range(lo + m, hi, m))
        top = ((1 << 50) - 1) // m * m + 1
        assert not any(inputs.is_prime(x) for x in range(allp[0] + m, top + 1, m))


def test_draws():
    g = inputs.rng(7, 0)
    s = inputs.ternary(g, 30000)
    assert set(np.unique(s)) == {-1, 0, 1} and abs(s.mean()) < 0.02
    e = inputs.rounded_gaussian(g, 200000)
    assert np.abs(e).max() <= 19 and abs(e.std() - 3.2) < 0.05
    q = [97, (1 << 50) - 27]
    u = inputs.uniform_residues(g, q, 5000, batch=2)
    assert u.shape == (2, 2, 5000) and (u[:, 0] < 97).all() and (u[:, 1] < q[1]).all()
    # same seed, same stream => same draws
    assert np.array_equal(inputs.ternary(inputs.rng(7, 3), 64), inputs.ternary(inputs.rng(7, 3), 64))


def test_feature_major_packing():
    x = np.arange(4 * 3, dtype=np.float64).reshape(4, 3)          # 4 tokens, 3... features must tile
    x = np.arange(8 * 4, dtype=np.float64).reshape(8, 4)          # 8 tokens, 4 features
    v = inputs.pack_feature_major(x, tokens_per_shard=4, slots=32)
    assert v.shape == (2, 32)
    T = 4
    for c in range(2):
        for f in range(4):
            for t in range(T):
                assert v[c, f * T + t] == x[c * T + t, f]
                assert v[c, 16 + f * T + t] == x[c * T + t, f]     # replicated block
