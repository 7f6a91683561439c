"""Pins for the checker's automorphism, ModUp, ModDown, rescale, key switch,
rotations and relinearised product -- exact big-integer statements on small
rings, decrypt-level statements on larger ones."""
import numpy as np
import pytest

from paper_2609_12378_b200 import inputs
from tests.harness import Client, centred, crt, params


def _coeff_ints(o, limbs_coeff, primes):
    """Per coefficient, the CRT integer of the given coefficient-domain limbs."""
    cols = np.asarray(limbs_coeff).T.tolist()
    return [crt(col, primes)[0] for col in cols]


@pytest.mark.parametrize("log_n", [3, 6, 10])
def test_automorphism_eval_equals_coefficient_definition(log_n):
    P = params(log_n, 2, 1, 2)
    o = P.oracle
    g = inputs.rng(41, log_n)
    a = inputs.uniform_residues(g, [o.mod[0]], P.N)[0]
    for gal in (5, 25, 3, 2 * P.N - 1, o.galois_element(3), o.galois_element(-1)):
        want = o.ntt(o.automorphism_coeff(a[0], gal, 0).reshape(1, -1))[0]
        assert np.array_equal(o.automorphism_eval(o.ntt(a)[0], gal), want)


def test_galois_element_is_left_rotation():
    """sigma_{5^r} on an encoded vector rotates the slots left by r (Eq. 5's rho^r)."""
    P = params(8, 2, 1, 2)
    o = P.oracle
    z = inputs.rng(42).uniform(-1, 1, P.n)
    m = o.encode_coeffs(z, 2.0 ** 40)
    for r in (1, 2, 7, P.n - 1, -3):
        assert o.galois_element(r) == pow(5, r % P.n, 2 * P.N)
        back = o.decode(o.automorphism_small(m, o.galois_element(r)).astype(np.longdouble), 2.0 ** 40).real
        assert np.abs(back - np.roll(z, -r)).max() < 1e-8


@pytest.mark.parametrize("log_n,L,K,dnum,level", [(4, 6, 2, 3, 6), (4, 6, 2, 3, 5), (4, 6, 2, 3, 2), (3, 4, 4, 1, 4), (5, 3, 1, 3, 3)])
def test_modup_big_integer(log_n, L, K, dnum, level):
    """Extended limbs = (d_c + u Q_j) mod t with one integer u per coefficient, |u| <= |D|/2."""
    P = params(log_n, L, K, dnum)
    o = P.oracle
    d = inputs.uniform_residues(inputs.rng(43, level), P.q[:level], P.N)[0]
    for j in range(o.num_digits(level)):
        lo, hi = j * o.alpha, min((j + 1) * o.alpha, level)
        ext = o.modup_digit(d, j)
        own = [int(x) for x in P.q[lo:hi]]
        targets = [int(x) for x in P.q[:level]] + [int(x) for x in P.p]
        assert ext.shape == (level + K, P.N)
        for k in range(P.N):
            v, Qj = crt(d[lo:hi, k], own)
            dc = centred(v, Qj)
            us = [u for u in range(-(hi - lo), hi - lo + 1)
                  if all((dc + u * Qj) % t == int(ext[x, k]) for x, t in enumerate(targets))]
            assert len(us) == 1 and 2 * abs(us[0]) <= hi - lo


@pytest.mark.parametrize("log_n,L,K,dnum,level", [(4, 6, 2, 3, 6), (4, 6, 2, 3, 3), (3, 4, 4, 1, 4), (5, 3, 1, 3, 2)])
def test_moddown_big_integer(log_n, L, K, dnum, level):
    """out = (U - r) / P exactly, r = U mod P in centred form up to v P with |v| <= K/2."""
    P = params(log_n, L, K, dnum)
    o = P.oracle
    primes = [int(x) for x in P.q[:level]] + [int(x) for x in P.p]
    g = inputs.rng(44, level)
    u_coeff = np.concatenate([inputs.uniform_residues(g, P.q[:level], P.N)[0], inputs.uniform_residues(g, P.p, P.N)[0]])
    u_eval = np.concatenate([o.ntt(u_coeff[:level]), o.ntt(u_coeff[level:], first=L)])
    out = o.intt(o.moddown(u_eval, level))
    Pp = 1
    for x in P.p:
        Pp *= int(x)
    Q = 1
    for x in P.q[:level]:
        Q *= int(x)
    for k in range(P.N):
        U, _ = crt(u_coeff[:, k], primes)
        o_int, _ = crt(out[:, k], primes[:level])
        r0 = centred(U % Pp, Pp)
        ok = [v for v in range(-K, K + 1) if (U - (r0 + v * Pp)) % Pp == 0 and ((U - (r0 + v * Pp)) // Pp - o_int) % Q == 0]
        assert ok and 2 * abs(ok[0]) <= K


@pytest.mark.parametrize("log_n,level", [(3, 2), (4, 4), (5, 3)])
def test_rescale_exact_rounding(log_n, level):
    """out = round(c / q_last) mod Q', per coefficient, exactly (no tie: q_last odd)."""
    P = params(log_n, 4, 1, 2)
    o = P.oracle
    primes = [int(x) for x in P.q[:level]]
    c_coeff = inputs.uniform_residues(inputs.rng(45, level), P.q[:level], P.N, batch=2)
    out = o.intt(o.rescale(o.ntt(c_coeff)))
    ql = primes[-1]
    Qp = 1
    for x in primes[:-1]:
        Qp *= x
    for comp in range(2):
        for k in range(P.N):
            cint, Q = crt(c_coeff[comp, :, k], primes)
            cc = centred(cint, Q)
            want = (2 * cc + ql) // (2 * ql)          # floor(c/q + 1/2) = nearest integer
            assert abs(want * ql - cc) * 2 < ql
            got, _ = crt(out[comp, :, k], primes[:-1])
            assert got == want % Qp


def _noise_after(cl, o, ct, want_coeffs):
    got = o.decrypt(ct, cl.s, exact=True)
    return max(abs(a - b) for a, b in zip(got, want_coeffs))


@pytest.mark.parametrize("log_n,L,K,dnum,level", [(10, 6, 2, 3, 6), (10, 6, 2, 3, 3), (10, 6, 1, 6, 6), (10, 4, 4, 1, 4)])
def test_keyswitch_decrypt_invariant(log_n, L, K, dnum, level):
    """k0 + k1 s = d s' + small, for s' = sigma_g(s) and s' = s^2."""
    P = params(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 51)
    d = inputs.uniform_residues(inputs.rng(46, level), P.q[:level], P.N)[0]
    gal = o.galois_element(5)
    for sprime_limbs, evk in (
        (o.small_to_limbs(o.automorphism_small(cl.s, gal), 0, level), cl.rotation_key(gal)),
        (None, cl.relin_key()),
    ):
        if sprime_limbs is None:
            sl = o.small_to_limbs(cl.s, 0, level)
            sprime_limbs = np.array([[int(a) * int(a) % o.mod[i] for a in sl[i].tolist()] for i in range(level)], dtype=np.uint64)
        k = o.keyswitch(d, evk)
        # want = d * s' as a "ciphertext" (d s', 0): compare decryptions
        ds = np.array([[int(a) * int(b) % o.mod[i] for a, b in zip(d[i].tolist(), sprime_limbs[i].tolist())] for i in range(level)], dtype=np.uint64)
        ref = np.stack([ds, np.zeros_like(ds)])
        diff = o.decrypt(_sub(o, k, ref), cl.s, exact=True)
        noise = max(abs(x) for x in diff)
        assert noise < 2 ** 14, noise          # ~ sqrt(beta N) sigma, nowhere near Q


def _sub(o, a, b):
    out = np.empty_like(a)
    for c in range(a.shape[0]):
        for i in range(a.shape[1]):
            m = o.mod[i]
            out[c, i] = (a[c, i].astype(object) - b[c, i].astype(object)) % m
    return out


@pytest.mark.parametrize("log_n,L,K,dnum,level", [(11, 6, 2, 3, 6), (11, 6, 2, 3, 4), (13, 6, 1, 6, 6)])
def test_rotate_decrypts_to_rotated_slots(log_n, L, K, dnum, level):
    P = params(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 52)
    z = inputs.rng(47, log_n).uniform(-1, 1, P.n)
    scale = 2.0 ** 40
    ct = cl.encrypt_slots(z, scale, level)
    rots = [1, 8, P.n - 5]
    gals = [o.galois_element(r) for r in rots]
    keys = [cl.rotation_key(g) for g in gals]
    hoisted = o.rotate_hoisted(ct, keys, gals)
    for i, r in enumerate(rots):
        plain = o.rotate(ct, keys[i], gals[i])
        want = np.roll(z, -r)
        zp, zh = cl.decrypt_slots(plain, scale), cl.decrypt_slots(hoisted[i], scale)
        assert np.abs(zp - want).max() < 2.0 ** -20
        assert np.abs(zh - want).max() < 2.0 ** -20
        assert np.abs(zp - zh).max() < 2.0 ** -20
        # slot 0 is where a constant rounding bias would show up (centred lifts keep it out)
        assert abs(zp[0] - want[0]) < 2.0 ** -22 and abs(zh[0] - want[0]) < 2.0 ** -22
    # rotate by r then by n - r returns the input slots
    back = o.rotate(o.rotate(ct, keys[0], gals[0]), cl.rotation_key(o.galois_element(-1)), o.galois_element(-1))
    assert np.abs(cl.decrypt_slots(back, scale) - z).max() < 2.0 ** -20


def test_hoisted_equals_plain_rotation_bit_for_bit():
    """ModUp's centred conversion is an odd function of the residue tuple, so it commutes with sigma_g (a signed
    permutation of coefficients): extending c1 once and permuting the digits gives the integers of the plain form."""
    for log_n, L, K, dnum, level, r in [(10, 6, 2, 3, 6, 3), (10, 6, 2, 3, 5, 1), (11, 4, 2, 2, 3, 100), (10, 4, 1, 4, 4, 7)]:
        P = params(log_n, L, K, dnum)
        o = P.oracle
        cl = Client(P, 53 + r)
        ct = cl.encrypt_slots(inputs.rng(48, r).uniform(-1, 1, P.n), 2.0 ** 40, level)
        gal = o.galois_element(r)
        key = cl.rotation_key(gal)
        assert np.array_equal(o.rotate(ct, key, gal), o.rotate_hoisted(ct, [key], [gal])[0])


def test_rotate_sum_pins():
    """A sum of rotations with one ModDown: n = 1 is rotate bit for bit; the extended-basis inner product is the
    big-integer sum of digit x key products; the result is ModDown of the summed inner products plus the permuted
    c0's (re-composed here from the separately pinned pieces); every coefficient differs from the sum of separate
    rotations by at most (n + 1) K / 2 (one conversion error instead of n); it decrypts to the sum of rotated slots."""
    log_n, L, K, dnum, level, n = 6, 6, 2, 3, 5, 4
    P = params(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 58)
    g = inputs.rng(58)
    scale = 2.0 ** 40
    zs = g.uniform(-1, 1, (n, P.n))
    rots = [1, 4, 9, P.n - 2]
    gals = [o.galois_element(r) for r in rots]
    keys = [cl.rotation_key(x) for x in gals]
    cts = np.stack([cl.encrypt_slots(z, scale, level) for z in zs])
    assert np.array_equal(o.rotate_sum(cts[:1], keys[:1], gals[:1]), o.rotate(cts[0], keys[0], gals[0]))
    out = o.rotate_sum(cts, keys, gals)
    primes = [int(x) for x in P.q[:level]] + [int(x) for x in P.p]
    kidx = list(range(level)) + [L + a for a in range(K)]
    U = np.zeros((2, level + K, P.N), dtype=object)
    z0 = np.zeros((level, P.N), dtype=object)
    for i in range(n):
        perm = np.stack([[o.automorphism_eval(cts[i][c][t], gals[i]) for t in range(level)] for c in range(2)])
        ext = o.modup_all(perm[1])
        u = o.inner_product(ext, keys[i])
        for c in range(2):
            for x, (m, kt) in enumerate(zip(primes, kidx)):
                want = sum(ext[j, x].astype(object) * keys[i][j, c, kt].astype(object) for j in range(ext.shape[0])) % m
                assert np.array_equal(u[c, x].astype(object), want)
                U[c, x] = (U[c, x] + want) % m
        z0 = z0 + perm[0].astype(object)
    q = np.array(primes[:level], dtype=object)[:, None]
    want0 = (o.moddown(U[0].astype(np.uint64), level).astype(object) + z0) % q
    assert np.array_equal(out[0].astype(object), want0)
    assert np.array_equal(out[1], o.moddown(U[1].astype(np.uint64), level))
    # against the sum of separate rotations, coefficient by coefficient
    sep = sum(o.rotate(cts[i], keys[i], gals[i]).astype(object) for i in range(n)) % q[None]
    diff = ((out.astype(object) - sep) % q[None]).astype(np.uint64)
    assert diff.any()
    for c in range(2):
        dc = o.intt(diff[c][None])[0]
        worst = max(abs(centred(*crt(dc[:, k], primes[:level]))) for k in range(P.N))
        assert worst <= (n + 1) * K / 2

    P = params(11, 6, 2, 3)
    o = P.oracle
    cl = Client(P, 59)
    zs = g.uniform(-1, 1, (3, P.n))
    rots = [8, 64, P.n - 16]
    gals = [o.galois_element(r) for r in rots]
    keys = [cl.rotation_key(x) for x in gals]
    for level in (6, 4):
        cts = np.stack([cl.encrypt_slots(z, scale, level) for z in zs])
        got = cl.decrypt_slots(o.rotate_sum(cts, keys, gals), scale)
        want = sum(np.roll(z, -r) for z, r in zip(zs, rots))
        assert np.abs(got - want).max() < 2.0 ** -20


@pytest.mark.parametrize("log_n,L,K,dnum,level", [(11, 6, 2, 3, 6), (11, 6, 2, 3, 3)])
def test_mul_relin_slot_product(log_n, L, K, dnum, level):
    P = params(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 54)
    g = inputs.rng(49)
    z, w = g.uniform(-1, 1, P.n), g.uniform(-1, 1, P.n)
    scale = 2.0 ** 40
    scale_b = float(P.q[level - 1])          # so that the rescale below lands back on 2^40 exactly
    ca, cb = cl.encrypt_slots(z, scale, level), cl.encrypt_slots(w, scale_b, level)
    rlk = cl.relin_key()
    out = o.mul_relin(ca, cb, rlk)
    assert np.abs(cl.decrypt_slots(out, scale * scale_b) - z * w).max() < 2.0 ** -20
    # three-component decrypt before relinearisation = two-component decrypt after, up to key-switch noise
    d3 = o.decrypt(o.tensor(ca, cb), cl.s, exact=True)
    d2 = o.decrypt(out, cl.s, exact=True)
    assert max(abs(x - y) for x, y in zip(d3, d2)) < 2 ** 16
    # then rescale: slots unchanged, scale divided by q_last
    rs = o.rescale(out)
    assert rs.shape[1] == level - 1
    assert np.abs(cl.decrypt_slots(rs, scale) - z * w).max() < 2.0 ** -20


def test_mul_relin_sum_pins():
    """Sum of products with one relinearisation: n = 1 is mul_relin bit for bit; the result is the key switch applied
    to the component-wise sum of the tensor products (checked against the separately exposed pieces); it decrypts
    to sum_i z_i w_i; and its exact decryption stays within key-switch noise of the three-component sum."""
    P = params(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, 57)
    g = inputs.rng(57)
    level, n, scale = 5, 6, 2.0 ** 40
    zs, ws = g.uniform(-1, 1, (n, P.n)), g.uniform(-1, 1, (n, P.n))
    ca = np.stack([cl.encrypt_slots(z, scale, level) for z in zs])
    cb = np.stack([cl.encrypt_slots(w, scale, level) for w in ws])
    rlk = cl.relin_key()
    assert np.array_equal(o.mul_relin_sum(ca[:1], cb[:1], rlk), o.mul_relin(ca[0], cb[0], rlk))
    out = o.mul_relin_sum(ca, cb, rlk)
    # the pieces: e = sum of tensor products modulo each prime, then mul_relin's own combination on e
    q = np.array(P.q[:level], dtype=object)[None, :, None]
    e = sum(o.tensor(ca[i], cb[i]).astype(object) for i in range(n)) % q
    e = e.astype(np.uint64)
    k = o.keyswitch(e[2], rlk)
    want = ((e[:2].astype(object) + k.astype(object)) % q).astype(np.uint64)
    assert np.array_equal(out, want)
    assert np.abs(cl.decrypt_slots(out, scale * scale) - (zs * ws).sum(0)).max() < 2.0 ** -20
    d3 = o.decrypt(e, cl.s, exact=True)
    d2 = o.decrypt(out, cl.s, exact=True)
    assert max(abs(x - y) for x, y in zip(d3, d2)) < 2 ** 16
    # and it is a different integer function from the sum of separately relinearised products (same plaintext)
    sep = sum(o.mul_relin(ca[i], cb[i], rlk).astype(object) for i in range(n)) % q
    assert not np.array_equal(sep.astype(np.uint64), out)
    assert np.abs(cl.decrypt_slots(sep.astype(np.uint64), scale * scale) - (zs * ws).sum(0)).max() < 2.0 ** -20


def test_const_ops_and_horner_pins():
    """Constant multiply / add are the plaintext operations with a constant-slot plaintext (checked against the
    encode + multiply-accumulate path and against decryption), and the Horner evaluation decrypts to the
    polynomial of the slots."""
    P = params(11, 8, 2, 4)
    o = P.oracle
    cl = Client(P, 58)
    g = inputs.rng(58)
    level = 8
    scale = float(2 ** 50)
    z = g.uniform(-1, 1, P.n)
    ct = cl.encrypt_slots(z, scale, level)
    # a constant-slot plaintext encodes to the constant polynomial round(c * scale): its limbs are that value everywhere
    c, cs = 0.37, float(P.q[level - 1])
    pt = o.encode(np.full(P.n, c), cs, level)
    v = int(np.rint(c * cs))
    assert all(np.all(pt[i] == np.uint64(v % P.q[i])) for i in range(level))
    assert np.array_equal(o.mul_const(ct, v), o.mul_plain_acc(ct, pt))
    assert np.array_equal(o.mul_const(ct, -v), o.mul_const(o.mul_const(ct, v), -1))
    assert np.abs(cl.decrypt_slots(o.mul_const(ct, v), scale * cs) - c * z).max() < 2.0 ** -30
    va = int(np.rint(-1.25 * scale))
    added = o.add_const(ct, va)
    assert np.array_equal(added[1], ct[1])
    assert np.abs(cl.decrypt_slots(added, scale) - (z - 1.25)).max() < 2.0 ** -30
    # Horner: degree 1 (no ciphertext product), 2 and 5
    rlk = cl.relin_key()
    for coeffs in ([0.5, -0.25], [0.1, 0.7, -0.3], [1.0, 1.0, 0.5, 1 / 6, 1 / 24, 1 / 120]):
        out, s_out = o.poly_eval(ct, scale, coeffs, rlk)
        assert out.shape[1] == level - (len(coeffs) - 1)
        want = sum(ck * z ** k for k, ck in enumerate(coeffs))
        assert np.abs(cl.decrypt_slots(out, s_out) - want).max() < 2.0 ** -25, coeffs


def test_poly_eval_tree_pins():
    """Log-depth polynomial evaluation: uses ceil(log2 d) + 1 levels, decrypts to the polynomial of the slots, and
    agrees with the Horner form (a different sequence of integer operations) to within the scheme's noise."""
    P = params(11, 8, 2, 4)
    o = P.oracle
    cl = Client(P, 59)
    z = inputs.rng(59).uniform(-1, 1, P.n)
    level, scale = 8, float(2 ** 50)
    ct = cl.encrypt_slots(z, scale, level)
    rlk = cl.relin_key()
    for coeffs in ([0.1, 0.7, -0.3], [1.0, 1.0, 0.5, 1 / 6, 1 / 24, 1 / 120], [0.0, 1.0, 0.0, -1 / 6, 0.0, 1 / 120, 0.0, -1 / 5040],
                   [0.3] + [(-1) ** k / (k + 1) for k in range(1, 16)]):
        d = len(coeffs) - 1
        out, so = o.poly_eval_tree(ct, scale, coeffs, rlk)
        assert out.shape[1] == level - ((d - 1).bit_length() + 1)
        want = sum(ck * z ** k for k, ck in enumerate(coeffs))
        got = cl.decrypt_slots(out, so)
        assert np.abs(got - want).max() < 2.0 ** -25, d
        if d <= 7:
            h, sh = o.poly_eval(ct, scale, coeffs, rlk)
            assert np.abs(cl.decrypt_slots(h, sh) - got).max() < 2.0 ** -25


def test_poly_eval_bsgs_pins():
    """Baby-step / giant-step polynomial evaluation: the polynomial of the slots (as poly_eval_tree's pin), the tree's
    result within noise, the level it ends on, and the special shapes (a block that is only a constant, zero coefficients,
    a degree that does not fill the last block)."""
    P = params(11, 9, 3, 3)
    o = P.oracle
    cl = Client(P, 81)
    g = inputs.rng(81)
    level, scale = 9, 2.0 ** 50
    z = g.uniform(-1, 1, P.n)
    ct = cl.encrypt_slots(z, scale, level)
    rlk = cl.relin_key()
    pv = np.polynomial.polynomial.polyval
    for d, m in [(15, 4), (9, 4), (7, 2), (31, 8), (5, 4)]:
        coeffs = g.uniform(-1, 1, d + 1) / (1 + np.arange(d + 1))
        if d == 15:
            coeffs[[5, 6, 7]] = 0.0          # block 1 is only a constant
            coeffs[9] = 0.0
        out, so = o.poly_eval_bsgs(ct, scale, coeffs, rlk, m)
        G = d // m + 1
        lb = level - max(m - 2, 0).bit_length()                       # level of x^(m-1)
        lg = level - (m - 1).bit_length() - max(G - 2, 0).bit_length()  # level of y^(G-1)
        assert out.shape[1] == min(lg, lb - 1) - 1
        got = cl.decrypt_slots(out, so).real
        assert np.abs(got - pv(z, coeffs)).max() < 2.0 ** -20, (d, m)
        if d <= 15:
            tree, st = o.poly_eval_tree(ct, scale, coeffs, rlk)
            assert np.abs(cl.decrypt_slots(tree, st).real - got).max() < 2.0 ** -22
