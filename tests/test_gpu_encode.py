"""GPU parity: encode, bit-exact against the CPU checker (same fp64 operation order)."""
import numpy as np
import pytest

from paper_2609_12378_b200 import binding, inputs
from tests.harness import params

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("log_n,L,K,dnum,batch,level,cplx", [
    (10, 4, 2, 2, 3, 4, False), (10, 4, 2, 2, 2, 1, True), (11, 4, 4, 1, 1, 3, True), (12, 3, 1, 3, 2, 3, False),
    (13, 6, 1, 6, 5, 6, False), (15, 3, 1, 3, 1, 2, True), (16, 24, 8, 3, 3, 24, False), (16, 24, 8, 3, 2, 7, True),
])
def test_encode_bit_exact(log_n, L, K, dnum, batch, level, cplx):
    from tests.gpu_util import context, dev, host
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    g = inputs.rng(301, log_n * 10 + level)
    re = g.uniform(-1, 1, (batch, P.n))
    im = g.normal(0, 0.3, (batch, P.n)) if cplx else None
    for scale in (2.0 ** 40, float(P.q[level - 1])):
        out = ctx.encode(dev(re), dev(im) if cplx else None, scale, level)
        got = host(out)
        for b in range(batch):
            z = re[b] + 1j * im[b] if cplx else re[b]
            assert np.array_equal(got[b], P.oracle.encode(z, scale, level)), (b, scale)
    assert ctx.encode_range_flag() == binding.OK


def test_encode_weight_like_and_decode():
    """Weights N(0, 0.02) replicated over tokens, as the projection encodes them."""
    from tests.gpu_util import context, dev, host
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    d = inputs.rng(302).normal(0, 0.02, 4096)
    z = np.repeat(d, 8)
    scale = float(P.q[23])
    got = host(ctx.encode(dev(z[None]), None, scale, 24))[0]
    assert np.array_equal(got, P.oracle.encode(z, scale, 24))
    coeffs = P.oracle.intt(got[:2])      # two limbs are enough to lift |m| < 2^62
    m = P.oracle.encode_coeffs(z, scale)
    q0 = int(P.q[0])
    assert [int(v) for v in coeffs[0][:64]] == [int(v) % q0 for v in m[:64]]
    back = P.oracle.decode(m.astype(np.longdouble), scale).real
    assert np.abs(back - z).max() < 2.0 ** -30


def test_encode_range_flag_and_errors():
    from tests.gpu_util import context, dev
    P, ctx = params(10, 4, 2, 2), context(10, 4, 2, 2)
    x = dev(np.full((1, P.n), 3.0))
    ctx.encode(x, None, 2.0 ** 62, 2)
    assert ctx.encode_range_flag() == binding.ERR_RANGE
    assert ctx.encode_range_flag() == binding.OK          # sticky until read, then cleared
    with pytest.raises(binding.CkksError) as e:
        ctx.encode(x, None, 2.0 ** 40, 5)
    assert e.value.code == binding.ERR_LEVEL
    lib = binding.load()
    out = dev(np.zeros((1, 2, P.N), dtype=np.uint64))
    assert lib.ckks_encode(ctx._h, x.data_ptr(), None, 1, 2.0 ** 40, 2, out.data_ptr(), None, 0, None) == binding.ERR_WORKSPACE
    assert lib.ckks_encode(ctx._h, x.data_ptr(), None, 1, -1.0, 2, out.data_ptr(), out.data_ptr(), 1 << 30, None) == binding.ERR_ARG
