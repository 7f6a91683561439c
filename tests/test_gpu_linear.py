"""GPU parity: the linear projection (Eq. 5, baby-step/giant-step), bit-exact on every
output limb against the CPU checker, and X W after decryption."""
import numpy as np
import pytest

from oracle.ckks_oracle import ProjDesc
from paper_2609_12378_b200 import binding, inputs
from tests.harness import Client, params

pytestmark = pytest.mark.gpu


def _run(log_n, L, K, dnum, level, d_in, d_out, T, S, B, seed, pt_scale=0.0, check_slots=True, lazy=False, compare=True):
    from tests.gpu_util import context, ct_dev, dev, host, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, seed)
    scale = 2.0 ** 40
    g = inputs.rng(seed, 1)
    X = inputs.activations_uniform(g, S * T, d_in)
    W = inputs.weights_normal(g, d_in, d_out, 0.02)
    desc = ProjDesc(d_in, d_out, T, S, B, pt_scale, lazy_moddown=lazy)
    F, ins, outs = o.proj_blocks(desc)
    cts = []
    for c in range(S):
        for (s0, mi) in ins:
            cts.append(cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T, s0:s0 + mi], T, o.n)[0], scale, level))
    rots = o.proj_rotations(desc)
    assert rots == ctx.linear_proj_rotations(d_in, d_out, T, S, B)
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    got = ctx.linear_proj([ct_dev(c, scale) for c in cts], dev(W), [key_dev(k, g_) for g_, k in keys.items()],
                          d_in, d_out, T, S, B, pt_scale, lazy_moddown=lazy)
    assert len(got) == S * len(outs)
    if not compare:
        return ctx, cts, keys
    want, want_scale = o.linear_proj(desc, np.stack(cts), W, keys, scale)
    Y = X @ W
    for i, ct in enumerate(got):
        arr = host(ct.data)
        assert ct.scale == want_scale and ct.level == level - 1
        assert np.array_equal(arr, want[i]), i
        if check_slots:
            c, ob = divmod(i, len(outs))
            o0, mo = outs[ob]
            sl = cl.decrypt_slots(arr, ct.scale).real.reshape(F, T)
            for r in range(0, F, max(1, F // 16)):
                assert np.abs(sl[r] - Y[c * T:(c + 1) * T, o0 + r % mo]).max() < (2.0 ** -17 if log_n >= 16 else 2.0 ** -20)
    return ctx, cts, keys


@pytest.mark.parametrize("d_in,d_out,T,S,B", [
    (16, 16, 32, 2, 4),      # square
    (16, 4, 32, 2, 2),       # wide with fold (K/V-like)
    (16, 24, 32, 1, 4),      # several output blocks, remainder output block (gate/up-like)
    (24, 16, 32, 2, 4),      # several input blocks, remainder input block (down-like)
    (8, 8, 32, 1, 8),        # replicated small block, single giant step
    (16, 16, 32, 1, 1),      # no baby rotations at all
])
def test_projection_shapes_small_ring(d_in, d_out, T, S, B):
    _run(10, 4, 2, 2, 4, d_in, d_out, T, S, B, seed=400 + d_in + d_out)


@pytest.mark.parametrize("d_in,d_out,T,S,B", [
    (64, 64, 8, 2, 32),      # J = 32: one k-step of the tensor-core multiply-accumulate
    (64, 64, 8, 3, 64),      # J = 64, odd shard count (column padding), single giant step
    (128, 64, 8, 1, 32),     # two input blocks: J = 64
    (64, 160, 8, 9, 32),     # remainder output block 32 | 64, folded; more than one column tile
    (96, 64, 8, 3, 32),      # remainder input block: the second block has one giant step, the first two
    (224, 64, 8, 2, 32),     # four input blocks (64, 64, 64, 32): four accumulating launches per group
])
def test_projection_tensor_core_mac_path(d_in, d_out, T, S, B):
    _run(10, 4, 2, 2, 4, d_in, d_out, T, S, B, seed=440 + d_in + d_out + S)


@pytest.mark.parametrize("d_in,d_out,T,S,B", [
    (16, 16, 32, 2, 4),      # three giant steps summed before one ModDown
    (16, 4, 32, 2, 2),       # followed by a fold
    (24, 16, 32, 2, 4),      # input blocks with different giant counts
    (8, 8, 32, 1, 8),        # no giant step to sum: the eager result
    (64, 160, 8, 9, 32),     # tensor-core path, several output blocks
    (224, 64, 8, 2, 32),     # four input blocks
])
def test_projection_lazy_moddown(d_in, d_out, T, S, B):
    """Giant steps summed in the key-switching basis, one ModDown per output ciphertext: bit-exact against the checker's
    variant of the schedule."""
    _run(10, 4, 2, 2, 4, d_in, d_out, T, S, B, seed=480 + d_in + d_out, lazy=True)


@pytest.mark.parametrize("log_n,L,K,dnum,level,d_in,d_out,T,S,B", [
    (10, 6, 2, 3, 5, 16, 16, 32, 2, 4),     # level below L, partial last digit
    (13, 6, 1, 6, 6, 64, 64, 32, 3, 8),     # six digits: the any-number-of-digits inner product, three shards
    (10, 4, 1, 4, 3, 16, 4, 32, 2, 2),      # one special prime, fold after the lazy sum
])
def test_projection_lazy_moddown_other_parameters(log_n, L, K, dnum, level, d_in, d_out, T, S, B):
    _run(log_n, L, K, dnum, level, d_in, d_out, T, S, B, seed=485 + log_n + dnum, lazy=True)


def test_projection_lazy_moddown_many_groups():
    """More giant steps than one group of accumulators holds (32 > 16): the running sum survives the next group's
    encode and multiply-accumulate."""
    _run(11, 4, 2, 2, 3, 128, 128, 8, 2, 4, seed=490, lazy=True)


@pytest.mark.parametrize("kernel", [binding.MAC_MMA_SPLIT, binding.MAC_MMA_ASYNC, binding.MAC_MMA_HALF, binding.MAC_TCGEN05])
def test_projection_tensor_core_mac_other_shapes(kernel):
    """The kernel's other forms (two warps per coefficient; the barrier-free pipeline; four coefficients per CTA; tcgen05
    with TMEM accumulators), selected by a context option, on a case with two k-steps, two column tiles and column
    padding."""
    from tests.gpu_util import context
    ctx = context(10, 4, 2, 2)
    ctx.set_option(binding.OPT_MAC_KERNEL, kernel)
    try:
        assert ctx.get_option(binding.OPT_MAC_KERNEL) == kernel
        _run(10, 4, 2, 2, 4, 64, 160, 8, 9, 32, seed=450)
        assert ctx.device_status() == 0
    finally:
        ctx.set_option(binding.OPT_MAC_KERNEL, binding.MAC_MMA)


def test_projection_with_tensor_core_basis_conversion():
    """ModUp's and ModDown's conversion matrices on the tensor cores (a context option): the same integers, on a shape
    with a fold, several output blocks and a partial last digit."""
    from tests.gpu_util import context
    ctxs = [context(10, 6, 2, 3), context(10, 4, 2, 2)]
    for c in ctxs:
        c.set_option(binding.OPT_CONV_KERNEL, binding.CONV_TENSOR)
    try:
        ctx, _, _ = _run(10, 6, 2, 3, 5, 16, 24, 32, 2, 4, seed=455)
        assert ctx.device_status() == 0
        _run(10, 4, 2, 2, 4, 64, 160, 8, 3, 32, seed=456, lazy=True)
    finally:
        for c in ctxs:
            c.set_option(binding.OPT_CONV_KERNEL, binding.CONV_FP64)


def test_options_reject_bad_values():
    from tests.gpu_util import context
    ctx = context(10, 4, 2, 2)
    for opt, bad in ((binding.OPT_NTT_FP_SHARE, 9), (binding.OPT_CONV_KERNEL, 2), (binding.OPT_MAC_KERNEL, 7), (binding.OPT_WAIT_CYCLES, -1),
                     (99, 0), (binding.OPT_STATIC_SCRATCH_BYTES, 1)):
        with pytest.raises(binding.CkksError) as e:
            ctx.set_option(opt, bad)
        assert e.value.code == binding.ERR_ARG
    assert ctx.get_option(99) == -1
    assert ctx.get_option(binding.OPT_WAIT_CYCLES) == 2_000_000_000
    assert ctx.get_option(binding.OPT_MAC_KERNEL) == binding.MAC_MMA and ctx.get_option(binding.OPT_CONV_KERNEL) == binding.CONV_FP64


def test_device_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """The mbarrier pipeline of the multiply-accumulate with a wait limit of zero cycles: the first wait that is not
    already satisfied (the operands of the first step are still on their way) gives up, the kernel waits for its own
    copies and returns, and the sticky flag is reported once.  With the limit restored the same call is bit-exact."""
    from tests.gpu_util import context
    ctx = context(10, 4, 2, 2)
    ctx.set_option(binding.OPT_MAC_KERNEL, binding.MAC_MMA_ASYNC)
    try:
        assert ctx.device_status() == binding.OK
        ctx.set_option(binding.OPT_WAIT_CYCLES, 0)
        _run(10, 4, 2, 2, 4, 64, 64, 8, 2, 32, seed=452, compare=False)
        assert ctx.device_status() == binding.ERR_TIMEOUT
        assert ctx.device_status() == binding.OK            # the flag was cleared by the query
        ctx.set_option(binding.OPT_WAIT_CYCLES, 2_000_000_000)
        _run(10, 4, 2, 2, 4, 64, 64, 8, 2, 32, seed=452)
        assert ctx.device_status() == binding.OK
    finally:
        ctx.set_option(binding.OPT_WAIT_CYCLES, 2_000_000_000)
        ctx.set_option(binding.OPT_MAC_KERNEL, binding.MAC_MMA)


def test_projection_multi_shares_baby_steps():
    """Three matrices on the same inputs (query/key/value-like: square, wide with fold, several output blocks):
    every output equals the checker's per-matrix result, and the shared call launches fewer kernels than three
    separate ones."""
    from tests.gpu_util import context, ct_dev, dev, host, key_dev
    log_n, L, K, dnum, level, d_in, T, S, B = 10, 4, 2, 2, 4, 16, 32, 2, 4
    d_outs = [16, 4, 24]
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 470)
    scale = 2.0 ** 40
    g = inputs.rng(470, 1)
    X = inputs.activations_uniform(g, S * T, d_in)
    Ws = [inputs.weights_normal(g, d_in, d_out, 0.02) for d_out in d_outs]
    descs = [ProjDesc(d_in, d_out, T, S, B, 0.0) for d_out in d_outs]
    F, ins, _ = o.proj_blocks(descs[0])
    cts = []
    for c in range(S):
        for (s0, mi) in ins:
            cts.append(cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T, s0:s0 + mi], T, o.n)[0], scale, level))
    rots = sorted(set(r for d in descs for r in o.proj_rotations(d)))
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    kd = [key_dev(k, g_) for g_, k in keys.items()]
    cd = [ct_dev(c, scale) for c in cts]
    n0 = binding.kernel_launches()
    got = ctx.linear_proj_multi(cd, [dev(W) for W in Ws], kd, d_in, d_outs, T, S, B)
    n_multi = binding.kernel_launches() - n0
    n_sep = 0
    for m, (d, W) in enumerate(zip(descs, Ws)):
        want, want_scale = o.linear_proj(d, np.stack(cts), W, keys, scale)
        assert len(got[m]) == len(want)
        for i, ct in enumerate(got[m]):
            assert ct.scale == want_scale and ct.level == level - 1
            assert np.array_equal(host(ct.data), want[i]), (m, i)
        n1 = binding.kernel_launches()
        ctx.linear_proj(cd, dev(W), kd, d_in, d_outs[m], T, S, B)
        n_sep += binding.kernel_launches() - n1
    assert n_multi < n_sep
    # the same call with the giant steps summed before one ModDown: every matrix equals the checker's lazy schedule
    got = ctx.linear_proj_multi(cd, [dev(W) for W in Ws], kd, d_in, d_outs, T, S, B, lazy_moddown=True)
    for m, (d_out, W) in enumerate(zip(d_outs, Ws)):
        want, _ = o.linear_proj(ProjDesc(d_in, d_out, T, S, B, 0.0, lazy_moddown=True), np.stack(cts), W, keys, scale)
        for i, ct in enumerate(got[m]):
            assert np.array_equal(host(ct.data), want[i]), (m, i)
    with pytest.raises(binding.CkksError) as e:       # unknown descriptor flags are refused
        bad = ctx._desc(16, 16, T, S, B)
        bad.flags = 2
        ws = ctx.workspace(1 << 20)
        ia = (binding.CCt * len(cd))(*[binding._cct(c) for c in cd])
        oa = (binding.CCt * 2)(*[binding._cct(ctx.empty_ct(level - 1)) for _ in range(2)])
        ka = (binding.CEvk * len(kd))(*[binding.CEvk(k.data.data_ptr(), k.galois) for k in kd])
        import ctypes as C
        ctx._check(binding.load().ckks_linear_proj(ctx._h, C.byref(bad), ia, dev(Ws[0]).data_ptr(), ka, len(kd), oa, ws.data_ptr(),
                                                   ws.numel(), None))
    assert e.value.code == binding.ERR_ARG
    with pytest.raises(binding.CkksError) as e:       # descriptors must share the input shape
        lib = binding.load()
        import ctypes as C
        da = (binding.CProjDesc * 2)(ctx._desc(16, 16, T, S, B), ctx._desc(16, 16, T, S, 2))
        ia = (binding.CCt * len(cd))(*[binding._cct(c) for c in cd])
        oa = (binding.CCt * 4)(*[binding._cct(ctx.empty_ct(level - 1)) for _ in range(4)])
        wa = (C.c_void_p * 2)(dev(Ws[0]).data_ptr(), dev(Ws[0]).data_ptr())
        ka = (binding.CEvk * len(kd))(*[binding.CEvk(k.data.data_ptr(), k.galois) for k in kd])
        ws = ctx.workspace(1 << 20)
        ctx._check(lib.ckks_linear_proj_multi(ctx._h, da, 2, ia, wa, ka, len(kd), oa, ws.data_ptr(), ws.numel(), None))
    assert e.value.code == binding.ERR_ARG


def test_projection_replays_from_a_cuda_graph():
    """The projection issues only stream work (kernels, device copies, memsets): captured once into a CUDA graph, it
    replays on new contents of the same buffers and returns what the direct call returns."""
    import torch
    from tests.gpu_util import context, ct_dev, dev, host, key_dev
    log_n, L, K, dnum, level, d_in, d_out, T, S, B = 10, 4, 2, 2, 4, 64, 64, 8, 2, 32
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, 495)
    scale = 2.0 ** 40
    g = inputs.rng(495, 1)
    W = dev(inputs.weights_normal(g, d_in, d_out, 0.02))
    desc = ProjDesc(d_in, d_out, T, S, B)
    keys = [key_dev(cl.rotation_key(o.galois_element(r)), o.galois_element(r)) for r in o.proj_rotations(desc)]

    def fresh():
        X = inputs.activations_uniform(g, S * T, d_in)
        return [cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T], T, o.n)[0], scale, level) for c in range(S)]
    first, second = fresh(), fresh()
    cts = [ct_dev(c, scale) for c in first]
    outs = [ctx.empty_ct(level - 1) for _ in range(S)]
    ws = torch.empty(ctx.linear_proj_workspace_bytes(d_in, d_out, T, S, B, level, True), dtype=torch.uint8, device="cuda")
    run = lambda: ctx.linear_proj(cts, W, keys, d_in, d_out, T, S, B, outs=outs, ws=ws, lazy_moddown=True)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()                                        # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run()
    for src in (second, first):
        for c, h in zip(cts, src):
            c.data.copy_(dev(h))
        graph.replay()
        replayed = [host(x.data).copy() for x in outs]
        run()
        for a, x in zip(replayed, outs):
            assert np.array_equal(a, host(x.data))
    assert ctx.device_status() == 0


def test_projection_explicit_pt_scale_and_lower_level():
    _run(10, 4, 2, 2, 3, 16, 16, 32, 1, 4, seed=410, pt_scale=2.0 ** 40, check_slots=False)


def test_projection_toy_config():
    """N = 2^13, 6 + 1 primes, dnum = 6, 32 tokens x 64 features times 64 x 64, B = G = 8."""
    ctx, cts, keys = _run(13, 6, 1, 6, 6, 64, 64, 32, 1, 8, seed=1001)
    assert len(keys) == 14


def test_projection_full_ring_small_shape():
    """N = 2^16, L = 24, dnum = 3 with 512 tokens per shard: F = 64 features, B = G = 8."""
    _run(16, 24, 8, 3, 24, 64, 64, 512, 1, 8, seed=420)


def test_projection_full_ring_tensor_core_mac():
    """N = 2^16, L = 24, dnum = 3, F = 64 features, B = 32, G = 2: the tensor-core multiply-accumulate at full ring size."""
    _run(16, 24, 8, 3, 24, 64, 64, 512, 2, 32, seed=421)


def test_projection_errors():
    from tests.gpu_util import context, ct_dev, dev, key_dev
    P, ctx = params(10, 4, 2, 2), context(10, 4, 2, 2)
    cl = Client(P, 430)
    ct = ct_dev(cl.encrypt_slots(np.zeros(P.n), 2.0 ** 40, 4), 2.0 ** 40)
    W = dev(np.zeros((16, 16)))
    with pytest.raises(binding.CkksError) as e:
        ctx.linear_proj([ct], W, [key_dev(np.zeros((2, 2, 6, P.N), dtype=np.uint64), 5)], 16, 16, 32, 1, 4)
    assert e.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as e:
        ctx.linear_proj_rotations(16, 16, 32, 1, 3)        # B must divide the diagonal count
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.CkksError) as e:
        ctx.linear_proj_rotations(12, 16, 32, 1, 4)        # remainder block 12 does not divide F = 16
    assert e.value.code == binding.ERR_UNSUPPORTED
