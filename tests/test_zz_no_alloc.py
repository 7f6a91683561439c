"""ckks_rescale_static: the rescale that brings its own scratch.

Callers that cannot allocate device memory when they need a rescale (inside a stream capture, behind a frozen
memory pool, or with only a fixed set of lent buffers) use this entry point; its scratch is a fixed array in
the library image.  The test calls it through the C ABI twice in a row on different inputs -- the second call
finds the first call's leftovers in the shared array -- and requires the same bytes as the ordinary
ckks_rescale, then checks that an input too large for the array is refused.  Collected last on purpose."""
import ctypes as C

import numpy as np
import pytest

from paper_2609_12378_b200 import binding, inputs
from tests.harness import params

pytestmark = pytest.mark.gpu


def _scratch_bytes(ctx):
    """The library's own limit (CKKS_STATIC_SCRATCH_BYTES of the build that is loaded)."""
    return ctx.get_option(binding.OPT_STATIC_SCRATCH_BYTES)


def _call_static(ctx, data, level, ncomp, scale, out):
    lib = binding.load()
    cin = binding.CCt(data.data_ptr(), level, ncomp, scale)
    cout = binding.CCt(out.data_ptr(), level - 1, ncomp, 0.0)
    rc = lib.ckks_rescale_static(ctx._h, C.byref(cin), C.byref(cout), None)
    return rc, cout


@pytest.mark.parametrize("log_n,L,K,dnum,level,ncomp", [(13, 6, 1, 6, 6, 2), (16, 24, 8, 3, 8, 2), (10, 6, 2, 3, 5, 1)])
def test_static_rescale_matches_rescale_twice(log_n, L, K, dnum, level, ncomp):
    import torch

    from tests.gpu_util import context, dev, host
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    assert ncomp * level * P.N * 8 <= _scratch_bytes(ctx)
    for call in range(2):
        x = inputs.uniform_residues(inputs.rng(900 + call, level), P.q[:level], P.N, ncomp)
        d = dev(x)
        want = ctx.rescale(binding.Ciphertext(d, 2.0 ** 80))
        out = torch.zeros((ncomp, level - 1, P.N), dtype=torch.uint64, device=d.device)
        rc, cout = _call_static(ctx, d, level, ncomp, 2.0 ** 80, out)
        assert rc == binding.OK
        assert cout.level == level - 1 and cout.ncomp == ncomp and cout.scale == want.scale
        got = host(out)
        assert np.array_equal(got, host(want.data)), call          # bit-exact, the tolerance of every integer test here
        assert np.array_equal(got, P.oracle.rescale(x)), call


def test_static_rescale_refuses_what_does_not_fit():
    import torch

    from tests.gpu_util import context, dev
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    level = 24                                                      # 2 * 24 * 65536 * 8 bytes = 24 MiB > 8 MiB
    d = dev(np.zeros((2, level, P.N), dtype=np.uint64))
    out = torch.zeros((2, level - 1, P.N), dtype=torch.uint64, device=d.device)
    rc, _ = _call_static(ctx, d, level, 2, 1.0, out)
    assert rc == binding.ERR_WORKSPACE
    assert b"built-in array" in binding.load().ckks_last_cuda_error(ctx._h)
    rc, _ = _call_static(ctx, d, 1, 2, 1.0, out)
    assert rc == binding.ERR_LEVEL
