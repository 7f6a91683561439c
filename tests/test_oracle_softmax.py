"""Pins for the checker's Softmax by doubling (Algorithm 1): against the same polynomial pipeline evaluated in the
clear (tight), against the true Softmax (as good as the synthetic polynomials), and the structure of the row sums."""
import numpy as np

from paper_2609_12378_b200 import inputs
from tests.harness import Client, params, softmax_case


def _keys(cl, o, row_len):
    keys, i = {}, 1
    while i < row_len:
        ge = o.galois_element(o.n // row_len * i)
        keys[ge] = cl.rotation_key(ge)
        i *= 2
    return keys


def test_softmax_doubling_matches_clear_pipeline_and_softmax():
    P = params(10, 17, 4, 5)
    o = P.oracle
    cl = Client(P, 71)
    row_len, rounds, level, scale = 16, 2, 17, 2.0 ** 50
    x, shift, ce, cr, clear, truth = softmax_case(P, 71, row_len, rounds)
    ct = cl.encrypt_slots(x, scale, level)
    out, so = o.softmax_doubling(ct, scale, shift, rounds, row_len, ce, cr, cl.relin_key(), _keys(cl, o, row_len))
    # exp tree: 3 levels; every round: square 1, inverse square root 3, two products 2
    assert out.shape[1] == level - 3 - rounds * 6
    got = cl.decrypt_slots(out, so).real
    assert np.abs(got - clear).max() < 2.0 ** -20
    assert np.abs(got - truth).max() < 0.05
    stride = P.n // row_len
    assert np.abs(got.reshape(row_len, stride).sum(0) - 1.0).max() < 0.1       # every row sums to about one


def test_softmax_doubling_with_block_polynomials():
    """The same loop with both polynomials (degree 8) evaluated by baby steps and giant steps: one round, the clear
    pipeline and the true Softmax again."""
    P = params(10, 13, 4, 4)
    o = P.oracle
    cl = Client(P, 73)
    row_len, rounds, level, scale = 16, 1, 13, 2.0 ** 50
    x, shift, ce, cr, clear, truth = softmax_case(P, 73, row_len, rounds, degree=8, spread=5.0)
    ct = cl.encrypt_slots(x, scale, level)
    out, so = o.softmax_doubling(ct, scale, shift, rounds, row_len, ce, cr, cl.relin_key(), _keys(cl, o, row_len), exp_m=4, rsqrt_m=4)
    assert out.shape[1] == level - 4 - 7
    got = cl.decrypt_slots(out, so).real
    assert np.abs(got - clear).max() < 2.0 ** -20
    assert np.abs(got - truth).max() < 0.02


def test_row_sum_by_strided_rotations():
    """The rotate-and-add ladder the Softmax rounds use: rotations by (n / R) 2^i leave the row sum in every slot of the row."""
    P = params(10, 4, 2, 2)
    o = P.oracle
    cl = Client(P, 72)
    R, level, scale = 8, 3, 2.0 ** 40
    stride = P.n // R
    z = inputs.rng(72, 1).uniform(-1, 1, P.n)
    s = cl.encrypt_slots(z, scale, level)
    i = 1
    while i < R:
        ge = o.galois_element(stride * i)
        s = o.add(s, o.rotate(s, cl.rotation_key(ge), ge))
        i *= 2
    want = np.tile(z.reshape(R, stride).sum(0), R)
    assert np.abs(cl.decrypt_slots(s, scale).real - want).max() < 2.0 ** -20
