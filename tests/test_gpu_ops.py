"""GPU parity: pointwise ops, rescale, rotations, relinearised product -- every RNS
integer output bit-exact against the CPU checker (so decrypted slots agree with the
checker's exactly, inside the 2^-20 bar); against the plaintext truth the slots are
within the scheme's own noise: 2^-20 up to N = 2^13, 2^-17 at N = 2^16 (Delta = 2^40)."""
import numpy as np
import pytest

from paper_2609_12378_b200 import binding, inputs
from tests.harness import Client, params

pytestmark = pytest.mark.gpu

SETS = [(10, 6, 2, 3), (11, 4, 4, 1), (13, 6, 1, 6), (16, 24, 8, 3)]


def truth_tol(log_n):
    return 2.0 ** -17 if log_n >= 16 else 2.0 ** -20


def _random_ct(P, level, seed, ncomp=2):
    return inputs.uniform_residues(inputs.rng(seed, level), P.q[:level], P.N, ncomp)


@pytest.mark.parametrize("log_n,L,K,dnum", SETS)
def test_mul_plain_acc_and_add(log_n, L, K, dnum):
    from tests.gpu_util import context, ct_dev, dev, host
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    for level in (L, 1):
        cts = [_random_ct(P, level, 200 + s) for s in range(3)]
        pt = inputs.uniform_residues(inputs.rng(210, level), P.q[:level], P.N)[0]
        pt2 = inputs.uniform_residues(inputs.rng(211, level), P.q[:level], P.N)[0]
        dcts = [ct_dev(c, 2.0 ** 40) for c in cts]
        accs = ctx.mul_plain_acc(dcts, binding.Plaintext(dev(pt), 2.0 ** 30))
        want = [o.mul_plain_acc(c, pt) for c in cts]
        for a, w in zip(accs, want):
            assert a.scale == 2.0 ** 70 and np.array_equal(host(a.data), w)
        ctx.mul_plain_acc(dcts[::-1], binding.Plaintext(dev(pt2), 2.0 ** 30), accs)
        for a, w, c in zip(accs, want, cts[::-1]):
            assert np.array_equal(host(a.data), o.mul_plain_acc(c, pt2, w.copy()))
        s = ctx.add(dcts[0], dcts[1])
        assert np.array_equal(host(s.data), o.add(cts[0], cts[1]))
        with pytest.raises(binding.CkksError) as e:
            ctx.mul_plain_acc(dcts, binding.Plaintext(dev(pt), 2.0 ** 31), accs)
        assert e.value.code == binding.ERR_SCALE


@pytest.mark.parametrize("log_n,L,K,dnum", SETS)
def test_rescale_bit_exact(log_n, L, K, dnum):
    from tests.gpu_util import context, ct_dev, host
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    for level in sorted({L, 2, max(2, L - 1)}):
        ct = _random_ct(P, level, 220)
        out = ctx.rescale(ct_dev(ct, 2.0 ** 80))
        assert out.level == level - 1 and out.scale == 2.0 ** 80 / float(P.q[level - 1])
        assert np.array_equal(host(out.data), P.oracle.rescale(ct))
    with pytest.raises(binding.CkksError) as e:
        ctx.rescale(ct_dev(_random_ct(P, 1, 221), 1.0))
    assert e.value.code == binding.ERR_LEVEL


@pytest.mark.parametrize("log_n,L,K,dnum,levels", [(10, 6, 2, 3, (6, 5, 2, 1)), (11, 4, 4, 1, (4, 3)), (13, 6, 1, 6, (6, 3)), (16, 24, 8, 3, (24, 17))])
def test_rotate_and_hoisted_bit_exact(log_n, L, K, dnum, levels):
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 230)
    rots = [1, 8, P.n - 3]
    gals = [o.galois_element(r) for r in rots]
    assert gals == [ctx.galois_element(r) for r in rots]
    keys = [cl.rotation_key(g) for g in gals]
    dkeys = [key_dev(k, g) for k, g in zip(keys, gals)]
    z = inputs.rng(231, log_n).uniform(-1, 1, P.n)
    for level in levels:
        ct = cl.encrypt_slots(z, 2.0 ** 40, level)
        dct = ct_dev(ct, 2.0 ** 40)
        for k, dk, g in zip(keys, dkeys, gals):
            out = ctx.rotate(dct, dk)
            assert np.array_equal(host(out.data), o.rotate(ct, k, g)), (level, g)
        plain = []
        for k, dk, g in zip(keys, dkeys, gals):
            plain.append(host(ctx.rotate(dct, dk).data))
        outs = ctx.rotate_hoisted(dct, dkeys)
        want = o.rotate_hoisted(ct, keys, gals)
        for i, out in enumerate(outs):
            got = host(out.data)
            assert np.array_equal(got, want[i]), (level, i)
            assert np.array_equal(got, plain[i]), (level, i)      # the contract: hoisted and plain rotation give the same integers
            if level >= 2:
                assert np.abs(cl.decrypt_slots(got, 2.0 ** 40).real - np.roll(z, -rots[i])).max() < truth_tol(log_n)
    # error paths: even Galois element, aliasing, short workspace
    bad = binding.SwitchKey(dkeys[0].data, 4)
    with pytest.raises(binding.CkksError) as e:
        ctx.rotate(dct, bad)
    assert e.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as e:
        ctx.rotate(dct, dkeys[0], out=dct)
    assert e.value.code == binding.ERR_ARG


@pytest.mark.parametrize("log_n,L,K,dnum,levels", [(10, 6, 2, 3, (6, 4, 1)), (13, 6, 1, 6, (6,)), (16, 24, 8, 3, (24,))])
def test_mul_relin_bit_exact(log_n, L, K, dnum, levels):
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 240)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    g = inputs.rng(241, log_n)
    z, w = g.uniform(-1, 1, P.n), g.uniform(-1, 1, P.n)
    for level in levels:
        sb = float(P.q[level - 1])
        ca, cb = cl.encrypt_slots(z, 2.0 ** 40, level), cl.encrypt_slots(w, sb, level)
        out = ctx.mul_relin(ct_dev(ca, 2.0 ** 40), ct_dev(cb, sb), drlk)
        got = host(out.data)
        assert out.scale == 2.0 ** 40 * sb
        assert np.array_equal(got, o.mul_relin(ca, cb, rlk)), level
        if level >= 2:
            assert np.abs(cl.decrypt_slots(got, out.scale) - z * w).max() < truth_tol(log_n)
            rs = ctx.rescale(out)
            assert np.abs(cl.decrypt_slots(host(rs.data), rs.scale) - z * w).max() < truth_tol(log_n)
    with pytest.raises(binding.CkksError) as e:
        ctx.mul_relin(ct_dev(ca, 1.0), ct_dev(cb, 1.0), binding.SwitchKey(drlk.data, 5))
    assert e.value.code == binding.ERR_NO_KEY


@pytest.mark.parametrize("log_n,L,K,dnum,level,n", [(10, 6, 2, 3, 5, 1), (10, 6, 2, 3, 6, 7), (11, 4, 2, 2, 3, 20), (16, 24, 8, 3, 24, 3)])
def test_mul_relin_sum_bit_exact(log_n, L, K, dnum, level, n):
    """Sum of n products with one relinearisation (n = 20 spans two launches of the accumulating kernel)."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 260 + n)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    g = inputs.rng(261, n)
    zs, ws = g.uniform(-1, 1, (n, P.n)), g.uniform(-1, 1, (n, P.n))
    sa, sb = 2.0 ** 40, 2.0 ** 38
    ca = np.stack([cl.encrypt_slots(z, sa, level) for z in zs])
    cb = np.stack([cl.encrypt_slots(w, sb, level) for w in ws])
    da, db = [ct_dev(c, sa) for c in ca], [ct_dev(c, sb) for c in cb]
    out = ctx.mul_relin_sum(da, db, drlk)
    got = host(out.data)
    assert out.scale == sa * sb and out.level == level
    assert np.array_equal(got, o.mul_relin_sum(ca, cb, rlk))
    assert np.abs(cl.decrypt_slots(got, out.scale) - (zs * ws).sum(0)).max() < truth_tol(log_n) * n
    if n == 1:
        assert np.array_equal(got, host(ctx.mul_relin(da[0], db[0], drlk).data))
    # errors: mixed scales, output aliasing an input, a rotation key instead of the relinearisation key
    if n > 1:
        with pytest.raises(binding.CkksError) as e:
            ctx.mul_relin_sum([da[0], binding.Ciphertext(da[1].data, 2.0 ** 39)], db[:2], drlk)
        assert e.value.code == binding.ERR_SCALE
    with pytest.raises(binding.CkksError) as e:
        ctx.mul_relin_sum(da, db, drlk, out=da[0])
    assert e.value.code == binding.ERR_ARG
    with pytest.raises(binding.CkksError) as e:
        ctx.mul_relin_sum(da, db, binding.SwitchKey(drlk.data, 5))
    assert e.value.code == binding.ERR_NO_KEY


@pytest.mark.parametrize("log_n,L,K,dnum,level,coeffs", [
    (11, 8, 2, 4, 8, [0.5, -0.25]),                                   # degree 1: no ciphertext product
    (11, 8, 2, 4, 8, [1.0, 1.0, 0.5, 1 / 6, 1 / 24, 1 / 120]),        # exp, degree 5
    (11, 8, 2, 4, 6, [0.1, 0.7, -0.3]),                               # below the top level
    (16, 24, 8, 3, 24, [0.0, 0.5, 0.0, -1 / 24, 0.0, 1 / 720, 0.0]),  # full ring, degree 6 with a zero leading coefficient
])
def test_const_ops_and_poly_eval_bit_exact(log_n, L, K, dnum, level, coeffs):
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 270)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    z = inputs.rng(271, log_n).uniform(-1, 1, P.n)
    scale = float(2 ** 50)
    ct = cl.encrypt_slots(z, scale, level)
    d = ct_dev(ct, scale)
    # constants
    cs = float(P.q[level - 1])
    m = ctx.mul_const(d, -0.37)
    assert m.scale == scale * cs and np.array_equal(host(m.data), o.mul_const(ct, int(np.rint(-0.37 * cs))))
    m2 = ctx.mul_const(d, 3.0, 2.0 ** 20)
    assert m2.scale == scale * 2.0 ** 20 and np.array_equal(host(m2.data), o.mul_const(ct, 3 << 20))
    a = ctx.add_const(d, 1.25)
    assert a.scale == scale and np.array_equal(host(a.data), o.add_const(ct, int(np.rint(1.25 * scale))))
    with pytest.raises(binding.CkksError) as e:
        ctx.add_const(d, 1.0e4)                  # 10^4 * 2^50 does not fit 2^62
    assert e.value.code == binding.ERR_RANGE
    # polynomial
    out = ctx.poly_eval(d, coeffs, drlk)
    want, want_scale = o.poly_eval(ct, scale, coeffs, rlk)
    assert out.level == level - (len(coeffs) - 1) and out.scale == want_scale
    got = host(out.data)
    assert np.array_equal(got, want)
    truth = sum(ck * z ** k for k, ck in enumerate(coeffs))
    assert np.abs(cl.decrypt_slots(got, out.scale) - truth).max() < 2.0 ** -22
    with pytest.raises(binding.CkksError) as e:
        ctx.poly_eval(d, [1.0] * (level + 1), drlk)          # degree = level: not enough limbs
    assert e.value.code == binding.ERR_LEVEL


@pytest.mark.parametrize("log_n,L,K,dnum,level,coeffs", [
    (11, 8, 2, 4, 8, [0.1, 0.7, -0.3]),
    (11, 8, 2, 4, 8, [0.0, 1.0, 0.0, -1 / 6, 0.0, 1 / 120, 0.0, -1 / 5040]),           # zero coefficients are skipped
    (11, 8, 2, 4, 7, [0.3] + [(-1) ** k / (k + 1) for k in range(1, 16)]),                # degree 15 in 5 levels
    (16, 24, 8, 3, 24, [1.0, 1.0, 0.5, 1 / 6, 1 / 24, 1 / 120, 1 / 720, 1 / 5040, 1 / 40320]),   # full ring, degree 8
])
def test_poly_eval_tree_bit_exact(log_n, L, K, dnum, level, coeffs):
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 280)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    z = inputs.rng(281, log_n).uniform(-1, 1, P.n)
    scale = float(2 ** 50)
    ct = cl.encrypt_slots(z, scale, level)
    out = ctx.poly_eval_tree(ct_dev(ct, scale), coeffs, drlk)
    want, want_scale = o.poly_eval_tree(ct, scale, coeffs, rlk)
    d = len(coeffs) - 1
    assert out.level == level - ((d - 1).bit_length() + 1) and out.scale == want_scale
    got = host(out.data)
    assert np.array_equal(got, want)
    truth = sum(ck * z ** k for k, ck in enumerate(coeffs))
    assert np.abs(cl.decrypt_slots(got, out.scale) - truth).max() < 2.0 ** -22
    with pytest.raises(binding.CkksError) as e:
        ctx.poly_eval_tree(ct_dev(ct, scale), [1.0] + [0.0] * d, drlk)
    assert e.value.code == binding.ERR_ARG


@pytest.mark.parametrize("log_n,L,K,dnum,level,n", [(10, 6, 2, 3, 6, 3), (11, 4, 2, 2, 3, 19), (16, 24, 8, 3, 24, 4)])
def test_mul_relin_batch_bit_exact(log_n, L, K, dnum, level, n):
    """n independent products with batched key switches (n = 19 spans two chunks): each equals mul_relin."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 290 + n)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    g = inputs.rng(291, n)
    ca = [cl.encrypt_slots(g.uniform(-1, 1, P.n), 2.0 ** 40, level) for _ in range(n)]
    cb = [cl.encrypt_slots(g.uniform(-1, 1, P.n), 2.0 ** 38, level) for _ in range(n)]
    outs = ctx.mul_relin_batch([ct_dev(c, 2.0 ** 40) for c in ca], [ct_dev(c, 2.0 ** 38) for c in cb], drlk)
    assert len(outs) == n
    for i in (range(n) if log_n < 16 else (0, n - 1)):
        assert outs[i].scale == 2.0 ** 78 and outs[i].level == level
        assert np.array_equal(host(outs[i].data), o.mul_relin(ca[i], cb[i], rlk)), i
    with pytest.raises(binding.CkksError) as e:
        ctx.mul_relin_batch([ct_dev(ca[0], 1.0)], [ct_dev(cb[0], 1.0)], binding.SwitchKey(drlk.data, 3))
    assert e.value.code == binding.ERR_NO_KEY


@pytest.mark.parametrize("log_n,L,K,dnum,level,n", [(10, 6, 2, 3, 5, 3), (11, 4, 2, 2, 4, 18), (16, 24, 8, 3, 24, 3)])
def test_rotate_batch_bit_exact(log_n, L, K, dnum, level, n):
    """One key, n ciphertexts, key switches side by side (n = 18 spans two chunks): each equals the plain rotation."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 300 + n)
    gal = o.galois_element(5)
    key = cl.rotation_key(gal)
    dkey = key_dev(key, gal)
    g = inputs.rng(301, n)
    cts = [cl.encrypt_slots(g.uniform(-1, 1, P.n), 2.0 ** 40, level) for _ in range(n)]
    outs = ctx.rotate_batch([ct_dev(c, 2.0 ** 40) for c in cts], dkey)
    for i in (range(n) if log_n < 16 else (0, n - 1)):
        assert outs[i].scale == 2.0 ** 40 and outs[i].level == level
        assert np.array_equal(host(outs[i].data), o.rotate(cts[i], key, gal)), i
    with pytest.raises(binding.CkksError) as e:
        ctx.rotate_batch([ct_dev(cts[0], 1.0)], binding.SwitchKey(dkey.data, 0))
    assert e.value.code == binding.ERR_NO_KEY


@pytest.mark.parametrize("log_n,L,K,dnum,level,n", [(10, 6, 2, 3, 5, 4), (11, 4, 2, 2, 4, 19), (10, 4, 1, 4, 3, 1), (10, 6, 1, 6, 6, 5), (16, 24, 8, 3, 24, 6)])
def test_rotate_sum_bit_exact(log_n, L, K, dnum, level, n):
    """sum_i rotate(ct_i, key_i) formed in the key-switching basis with one ModDown (n = 19 spans two chunks; n = 1 is the
    plain rotation)."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 310 + n)
    rots = [1 + 3 * i for i in range(min(n, 5))]
    gals = [o.galois_element(r) for r in rots]
    hk = [cl.rotation_key(x) for x in gals]
    dk = [key_dev(k, x) for k, x in zip(hk, gals)]
    g = inputs.rng(311, n)
    cts = np.stack([cl.encrypt_slots(g.uniform(-1, 1, P.n), 2.0 ** 40, level) for _ in range(n)])
    pick = [i % len(rots) for i in range(n)]
    out = ctx.rotate_sum([ct_dev(c, 2.0 ** 40) for c in cts], [dk[j] for j in pick])
    assert out.scale == 2.0 ** 40 and out.level == level
    assert np.array_equal(host(out.data), o.rotate_sum(cts, [hk[j] for j in pick], [gals[j] for j in pick]))
    if n == 1:
        assert np.array_equal(host(out.data), o.rotate(cts[0], hk[0], gals[0]))
    # in place on one of the inputs
    d = [ct_dev(c, 2.0 ** 40) for c in cts]
    ctx.rotate_sum(d, [dk[j] for j in pick], out=d[-1])
    assert np.array_equal(host(d[-1].data), host(out.data))
    with pytest.raises(binding.CkksError) as e:
        ctx.rotate_sum(d[:1], [binding.SwitchKey(dk[0].data, 0)])
    assert e.value.code == binding.ERR_NO_KEY


@pytest.mark.parametrize("log_n,d,m", [(11, 15, 4), (11, 9, 4), (11, 7, 2), (11, 31, 8), (11, 5, 4), (16, 31, 8)])
def test_poly_eval_bsgs_bit_exact(log_n, d, m):
    """Baby-step / giant-step polynomial evaluation: the checker's integers (constant-only block and zero coefficients at
    degree 15; a partial last block; N = 2^16 at level 24) and the error paths."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    cfg = (11, 9, 3, 3) if log_n == 11 else (16, 24, 8, 3)
    P, ctx = params(*cfg), context(*cfg)
    o = P.oracle
    cl = Client(P, 81)
    g = inputs.rng(81, d)
    level, scale = cfg[1], 2.0 ** 50
    z = g.uniform(-1, 1, P.n)
    ct = cl.encrypt_slots(z, scale, level)
    rlk = cl.relin_key()
    coeffs = g.uniform(-1, 1, d + 1) / (1 + np.arange(d + 1))
    if d == 15:
        coeffs[[5, 6, 7]] = 0.0
        coeffs[9] = 0.0
    want, so = o.poly_eval_bsgs(ct, scale, coeffs, rlk, m)
    got = ctx.poly_eval_bsgs(ct_dev(ct, scale), coeffs, m, key_dev(rlk, 0))
    assert got.level == want.shape[1] and got.scale == so
    arr = host(got.data)
    assert np.array_equal(arr, want)
    assert np.abs(cl.decrypt_slots(arr, so).real - np.polynomial.polynomial.polyval(z, coeffs)).max() < 2.0 ** -20
    if d == 15:
        for bad_m in (3, 16, 1):
            with pytest.raises(binding.CkksError) as e:
                ctx.poly_eval_bsgs(ct_dev(ct, scale), coeffs, bad_m, key_dev(rlk, 0))
            assert e.value.code == binding.ERR_ARG
        with pytest.raises(binding.CkksError) as e:
            ctx.poly_eval_bsgs(ct_dev(ct[:, :3], scale), coeffs, 4, key_dev(rlk, 0))
        assert e.value.code == binding.ERR_LEVEL


def test_poly_eval_bsgs_batch_bit_exact():
    """The same polynomial of several ciphertexts, spread over the context's lanes: every output equals the checker's
    evaluation of its own input (seven ciphertexts on four lanes, then on one)."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    cfg = (11, 9, 3, 3)
    P, ctx = params(*cfg), context(*cfg)
    o = P.oracle
    cl = Client(P, 83)
    g = inputs.rng(83, 2)
    level, scale, d, m = 9, 2.0 ** 50, 15, 4
    coeffs = g.uniform(-1, 1, d + 1) / (1 + np.arange(d + 1))
    rlk = cl.relin_key()
    cts = [cl.encrypt_slots(g.uniform(-1, 1, P.n), scale, level) for _ in range(7)]
    want = [o.poly_eval_bsgs(c, scale, coeffs, rlk, m) for c in cts]
    dev = [ct_dev(c, scale) for c in cts]
    try:
        for lanes in (4, 1):
            ctx.set_option(binding.OPT_LANES, lanes)
            got = ctx.poly_eval_bsgs_batch(dev, coeffs, m, key_dev(rlk, 0))
            for x, (w, so) in zip(got, want):
                assert x.level == w.shape[1] and x.scale == so and np.array_equal(host(x.data), w)
    finally:
        ctx.set_option(binding.OPT_LANES, 4)
    assert ctx.device_status() == binding.OK
    with pytest.raises(binding.CkksError) as e:
        ctx.poly_eval_bsgs_batch(dev, coeffs, 3, key_dev(rlk, 0))
    assert e.value.code == binding.ERR_ARG


def test_softmax_by_doubling_bit_exact():
    """Algorithm 1 with synthetic polynomials on 32 rows of 16 scores (two rounds, degree 4): the composite entry point
    returns the checker's integers, which decrypt to the same pipeline in the clear and to the Softmax of every row."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    from tests.harness import softmax_case
    P, ctx = params(10, 17, 4, 5), context(10, 17, 4, 5)
    o = P.oracle
    cl = Client(P, 71)
    row_len, rounds, level, scale = 16, 2, 17, 2.0 ** 50
    x, shift, ce, cr, clear, truth = softmax_case(P, 71, row_len, rounds)
    ct = cl.encrypt_slots(x, scale, level)
    rlk = cl.relin_key()
    keys, i = {}, 1
    while i < row_len:
        ge = o.galois_element(P.n // row_len * i)
        keys[ge] = cl.rotation_key(ge)
        i *= 2
    want, want_scale = o.softmax_doubling(ct, scale, shift, rounds, row_len, ce, cr, rlk, keys)
    got = ctx.softmax(ct_dev(ct, scale), shift, rounds, row_len, ce, cr, key_dev(rlk, 0), [key_dev(k, g) for g, k in keys.items()])
    assert got.level == want.shape[1] == 2 and got.scale == want_scale
    arr = host(got.data)
    assert np.array_equal(arr, want)
    slots = cl.decrypt_slots(arr, got.scale).real
    assert np.abs(slots - clear).max() < 2.0 ** -20 and np.abs(slots - truth).max() < 0.05
    with pytest.raises(binding.CkksError) as e:          # a rotation key of the ladder is missing
        ctx.softmax(ct_dev(ct, scale), shift, rounds, row_len, ce, cr, key_dev(rlk, 0), [key_dev(k, g) for g, k in list(keys.items())[1:]])
    assert e.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as e:          # not enough levels for the rounds
        ctx.softmax(ct_dev(ct[:, :10], scale), shift, rounds, row_len, ce, cr, key_dev(rlk, 0), [key_dev(k, g) for g, k in keys.items()])
    assert e.value.code == binding.ERR_LEVEL


def test_softmax_without_rounds_is_the_exponential_polynomial():
    """rounds = 0: the shift and p_exp only, i.e. poly_eval_tree of x - shift; no rotation key is needed."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(10, 6, 2, 3), context(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, 74)
    level, scale, shift = 6, 2.0 ** 50, 1.5
    z = inputs.rng(74, 1).uniform(-1, 1, P.n)
    ct = cl.encrypt_slots(z, scale, level)
    rlk = cl.relin_key()
    coeffs = [1.0, 0.5, 0.125, 0.02, 0.003]
    want, ws = o.softmax_doubling(ct, scale, shift, 0, 16, coeffs, [], rlk, {})
    tree, ts = o.poly_eval_tree(o.add_const(ct, int(np.rint(-shift * scale))), scale, coeffs, rlk)
    assert np.array_equal(want, tree) and ws == ts
    got = ctx.softmax(ct_dev(ct, scale), shift, 0, 16, coeffs, [], key_dev(rlk, 0), [])
    assert got.scale == ws and np.array_equal(host(got.data), want)


def test_rotate_batch_in_place():
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(10, 6, 2, 3), context(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, 320)
    gal = o.galois_element(7)
    key = cl.rotation_key(gal)
    g = inputs.rng(321, 1)
    cts = [cl.encrypt_slots(g.uniform(-1, 1, P.n), 2.0 ** 40, 4) for _ in range(3)]
    d = [ct_dev(c, 2.0 ** 40) for c in cts]
    ctx.rotate_batch(d, key_dev(key, gal), outs=d)
    for i in range(3):
        assert np.array_equal(host(d[i].data), o.rotate(cts[i], key, gal))


def test_softmax_with_block_polynomials_bit_exact():
    """One round with degree-8 polynomials evaluated by baby steps and giant steps (blocks of 4)."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    from tests.harness import softmax_case
    P, ctx = params(10, 13, 4, 4), context(10, 13, 4, 4)
    o = P.oracle
    cl = Client(P, 73)
    row_len, rounds, level, scale = 16, 1, 13, 2.0 ** 50
    x, shift, ce, cr, clear, truth = softmax_case(P, 73, row_len, rounds, degree=8, spread=5.0)
    ct = cl.encrypt_slots(x, scale, level)
    rlk = cl.relin_key()
    keys, i = {}, 1
    while i < row_len:
        ge = o.galois_element(P.n // row_len * i)
        keys[ge] = cl.rotation_key(ge)
        i *= 2
    want, want_scale = o.softmax_doubling(ct, scale, shift, rounds, row_len, ce, cr, rlk, keys, exp_m=4, rsqrt_m=4)
    got = ctx.softmax(ct_dev(ct, scale), shift, rounds, row_len, ce, cr, key_dev(rlk, 0), [key_dev(k, g) for g, k in keys.items()],
                      exp_m=4, rsqrt_m=4)
    assert got.level == want.shape[1] and got.scale == want_scale
    assert np.array_equal(host(got.data), want)


def test_repeatability():
    """Same call twice gives the same bytes (a race would show up as a difference)."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(13, 6, 1, 6), context(13, 6, 1, 6)
    cl = Client(P, 250)
    g = P.oracle.galois_element(5)
    dk = key_dev(cl.rotation_key(g), g)
    dct = ct_dev(cl.encrypt_slots(np.ones(P.n), 2.0 ** 40, 6), 2.0 ** 40)
    a = host(ctx.rotate(dct, dk).data).copy()
    for _ in range(3):
        assert np.array_equal(host(ctx.rotate(dct, dk).data), a)
