"""GPU parity: batched NTT / inverse NTT, bit-exact against the CPU checker."""
import numpy as np
import pytest

from paper_2609_12378_b200 import binding, inputs
from tests.harness import params

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("log_n,L,K,dnum,batch,first,nl", [
    (10, 4, 2, 2, 3, 0, 4), (10, 4, 2, 2, 1, 3, 3), (11, 6, 2, 3, 2, 6, 2), (12, 3, 1, 3, 5, 1, 3),
    (13, 6, 1, 6, 2, 0, 7), (14, 3, 1, 3, 1, 0, 4), (15, 3, 1, 3, 2, 2, 2), (16, 24, 8, 3, 2, 20, 9),
])
def test_ntt_bit_exact(log_n, L, K, dnum, batch, first, nl):
    from tests.gpu_util import context, dev, host
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    x = inputs.uniform_residues(inputs.rng(101, log_n), P.oracle.mod[first:first + nl], P.N, batch)
    d = dev(x)
    ctx.ntt(d, first)
    want = P.oracle.ntt(x, first)
    assert np.array_equal(host(d), want)
    ctx.intt(d, first)
    assert np.array_equal(host(d), x)
    # inverse alone, from the checker's forward output
    d2 = dev(want)
    ctx.intt(d2, first)
    assert np.array_equal(host(d2), x)


def test_ntt_edge_values():
    """All-zero, all q-1, delta and X: closed forms NTT(1) = 1, NTT(X)[p] = psi^(2 brev(p) + 1)."""
    from tests.gpu_util import context, dev, host
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    N, mods = P.N, P.oracle.mod
    x = np.zeros((4, 32, N), dtype=np.uint64)
    x[1] = (np.array(mods, dtype=np.uint64) - 1)[:, None]
    x[2, :, 0] = 1
    x[3, :, 1] = 1
    d = dev(x)
    ctx.ntt(d, 0)
    got = host(d)
    assert (got[0] == 0).all() and (got[2] == 1).all()
    assert np.array_equal(got, P.oracle.ntt(x, 0))
    assert [int(v) for v in got[3, :, 0]] == [P.oracle.root(t) for t in range(32)]   # brev(0) = 0 -> psi^1


def test_ntt_microbench_config_full_size():
    """N = 2^16, 24 limbs, batch 32 (the NTT microbenchmark configuration): forward vs checker, round trip."""
    from tests.gpu_util import context, dev, host
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    x = inputs.uniform_residues(inputs.rng(1002, 0), P.q, P.N, 32)
    d = dev(x)
    ctx.ntt(d, 0)
    assert np.array_equal(host(d), P.oracle.ntt(x, 0))
    ctx.intt(d, 0)
    assert np.array_equal(host(d), x)


def test_ntt_argument_errors():
    from tests.gpu_util import context, dev
    ctx = context(10, 4, 2, 2)
    d = dev(np.zeros((1, 4, 1024), dtype=np.uint64))
    with pytest.raises(binding.CkksError) as e:
        ctx.ntt(d, 4)            # primes 4..7 do not exist (L + K = 6)
    assert e.value.code == binding.ERR_LEVEL
    lib = binding.load()
    assert lib.ckks_ntt(ctx._h, None, 1, 0, 1, None) == binding.ERR_ARG
    assert lib.ckks_intt(ctx._h, d.data_ptr(), 0, 0, 1, None) == binding.ERR_ARG


def test_butterfly_probe_counts_and_errors():
    """The register-resident butterfly kernel (measurement aid): launch count and argument checks."""
    import torch
    from tests.gpu_util import context
    ctx = context(16, 24, 8, 3)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    scratch = torch.zeros(sms * 1024, dtype=torch.int64, device="cuda").view(torch.uint64)
    assert ctx.ntt_butterfly_probe(8, scratch) == sms * 3 * 256 * 8 * 32
    torch.cuda.synchronize()
    assert int(scratch.view(torch.int64).abs().sum()) == 0          # the sink is never written
    with pytest.raises(binding.CkksError) as e:
        ctx.ntt_butterfly_probe(8, scratch[:16])
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.CkksError) as e:
        context(10, 4, 2, 2).ntt_butterfly_probe(8, scratch)
    assert e.value.code == binding.ERR_UNSUPPORTED
