"""Parity of the CUDA kernels with the CPU oracle, kernel by kernel, through the C-ABI.

Integer, byte and scale-bit-pattern work must be bit-exact; dequantized fp32 outputs whose
operation order is pinned (rescale, ReLU) must be bit-exact too (tolerance 1e-6 relative is
slack); GELU outputs within 1e-6 relative with a floor of 1e-6 * max|y|; SSE within 1e-5
relative with identical rankings; bf16 layers within 1e-2 (normwise) of the fp64 reference.
"""
import numpy as np
import pytest
import torch

from oracle import qcfg_oracle as orc

pytestmark = pytest.mark.gpu

BITS = list(range(2, 9))


@pytest.fixture(scope="module")
def ctx():
    import paper_2302_01382_b200 as q
    c = q.Context(0)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


# ----------------------------------------------------------------------------- absmax, scales

@pytest.mark.parametrize("shape", [(1, 1), (7, 13), (64, 256), (300, 768), (10, 147), (1025, 1000), (5, 40000)])
def test_absmax_matches_oracle(ctx, shape):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(shape[0] * 1000 + shape[1])
    x = (rng.standard_normal(shape) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
    xd = dev(x)
    np.testing.assert_array_equal(host(ctx.calibrate(xd, q.PER_TENSOR))[0], orc.absmax(x))
    np.testing.assert_array_equal(host(ctx.calibrate(xd, q.PER_ROW)), orc.absmax(x, orc.PER_ROW))
    if shape[1] > 8:  # strided, unaligned view
        v = xd[:, 3:shape[1] - 1]
        np.testing.assert_array_equal(host(ctx.calibrate(v, q.PER_TENSOR))[0], orc.absmax(x[:, 3:shape[1] - 1]))
        np.testing.assert_array_equal(host(ctx.calibrate(v, q.PER_ROW)), orc.absmax(x[:, 3:shape[1] - 1], orc.PER_ROW))
    ctx.check_sync()


def test_absmax_propagates_nonfinite_and_empty(ctx):
    import paper_2302_01382_b200 as q
    x = np.ones((4, 64), np.float32)
    x[2, 5] = np.nan
    assert not np.isfinite(host(ctx.calibrate(dev(x), q.PER_TENSOR))[0])
    x[2, 5] = -np.inf
    assert np.isinf(host(ctx.calibrate(dev(x), q.PER_ROW))[2])
    z = torch.zeros((3, 8), device="cuda")
    assert host(ctx.calibrate(z, q.PER_TENSOR))[0] == 0


@pytest.mark.parametrize("b", BITS)
def test_scales_bit_patterns(ctx, b):
    rng = np.random.default_rng(b)
    A = np.concatenate([(10.0 ** rng.uniform(-30, 30, 4000)).astype(np.float32), np.zeros(3, np.float32)])
    s, inv = ctx.scales_from_absmax(dev(A), b)
    so, io = orc.scales_from_absmax(A, b)
    np.testing.assert_array_equal(host(s).view(np.uint32), so.view(np.uint32))
    np.testing.assert_array_equal(host(inv).view(np.uint32), io.view(np.uint32))


# ----------------------------------------------------------------------------- quantize

@pytest.mark.parametrize("b", BITS)
@pytest.mark.parametrize("shape", [(3, 5), (64, 256), (257, 147), (130, 1000)])
def test_quantize_codes_bit_exact(ctx, b, shape):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(b * 100 + shape[1])
    x = rng.standard_normal(shape).astype(np.float32)
    # exact ties and values beyond the calibrated range
    x[0, :min(5, shape[1])] = (np.arange(min(5, shape[1])) + 0.5).astype(np.float32)
    xd = dev(x)
    # per row, own maxima
    A = orc.absmax(x, orc.PER_ROW)
    so, io = orc.scales_from_absmax(A, b)
    codes = host(ctx.quantize(xd, dev(io), q.PER_ROW, b))
    np.testing.assert_array_equal(codes[:, :shape[1]], orc.quantize(x, io[:, None], b))
    assert not codes[:, shape[1]:].any()
    # per tensor, a calibrated maximum smaller than the data (live clip)
    At = np.float32(orc.absmax(x) * 0.37)
    st, it = orc.scales_from_absmax(At, b)
    codes = host(ctx.quantize(xd, dev(np.array([it], np.float32)), q.PER_TENSOR, b))
    want = orc.quantize(x, it, b)
    np.testing.assert_array_equal(codes[:, :shape[1]], want)
    assert np.abs(want).max() == orc.qmax(b)


def test_quantize_bf16_bit_exact(ctx):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(0)
    x = (rng.standard_normal((77, 203)) * 10.0 ** rng.uniform(-5, 5, (77, 1))).astype(np.float32)
    out = ctx.quantize(dev(x), None, q.PER_TENSOR, 16)
    got = host(out.float())[:, :203]
    np.testing.assert_array_equal(got.view(np.uint32), orc.bf16_round(x).view(np.uint32))


# ----------------------------------------------------------------------------- sweep

SWEEP_SHAPES = [(256, 256), (10, 256), (768, 768), (300, 3072), (97, 1024), (33, 4096), (64, 147), (128, 576),
                (40, 4608), (5, 8192), (3, 9000), (17, 64), (1, 4), (2500, 32)]


def _check_sweep(ctx, tensors, granularity):
    sse, amax = ctx.quant_error_sweep([dev(t) for t in tensors], granularity)
    ctx.check_sync()
    sse, amax = host(sse), host(amax)
    so, ao = orc.quant_error_sweep(tensors, granularity)
    np.testing.assert_array_equal(amax, ao)
    np.testing.assert_allclose(sse, so, rtol=1e-5, atol=0)
    sizes = [t.size for t in tensors]
    eg, eo = orc.e_qe_table(sse, sizes, amax), orc.e_qe_table(so, sizes, ao)
    for j in range(7):
        rg, ro = orc.ranking(eg[:, j]), orc.ranking(eo[:, j])
        if not np.array_equal(rg, ro):   # only near-ties may swap
            for a, b in zip(rg, ro):
                assert a == b or abs(eo[a, j] - eo[b, j]) <= 1e-5 * eo[a, j]


@pytest.mark.parametrize("granularity", [orc.PER_ROW, orc.PER_TENSOR])
def test_sweep_matches_oracle(ctx, granularity):
    rng = np.random.default_rng(42)
    tensors = []
    for i, s in enumerate(SWEEP_SHAPES):
        w = (rng.standard_normal(s) * 0.02).astype(np.float32)
        w[rng.random(s) < 1e-3] *= 20
        if i % 3 == 0:
            w *= rng.uniform(0.2, 5, (s[0], 1)).astype(np.float32)
        tensors.append(w)
    tensors.append(np.zeros((8, 64), np.float32))
    _check_sweep(ctx, tensors, granularity)


def test_sweep_is_deterministic_and_handles_subranges(ctx):
    rng = np.random.default_rng(1)
    ts = [dev((rng.standard_normal((500, 768)) * 0.02).astype(np.float32)) for _ in range(3)]
    a, _ = ctx.quant_error_sweep(ts)
    b, _ = ctx.quant_error_sweep(ts)
    assert torch.equal(a, b)
    c, _ = ctx.quant_error_sweep(ts, b_lo=4, b_hi=6)
    assert torch.equal(c, a[:, 2:5])


# ----------------------------------------------------------------------------- GEMM

def _codes(rng, rows, k, ld, lo=-127, hi=127):
    q = np.zeros((rows, ld), np.int8)
    q[:, :k] = rng.integers(lo, hi + 1, (rows, k), dtype=np.int8)
    return q


GEMM_SHAPES = [(64, 16, 32), (128, 32, 128), (64, 10, 256), (300, 200, 150), (700, 1000, 528), (129, 257, 3072),
               (1000, 768, 768), (260, 2304, 144), (3, 5, 7), (2048, 64, 64), (512, 512, 4608)]


@pytest.mark.parametrize("m,n,k", GEMM_SHAPES)
def test_gemm_i8_accumulators_and_rescale_bit_exact(ctx, m, n, k):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(m + n + k)
    ld = (k + 15) // 16 * 16
    qx, qw = _codes(rng, m, k, ld), _codes(rng, n, k, ld)
    sw = (10.0 ** rng.uniform(-4, -2, n)).astype(np.float32)
    sx = np.float32(0.0173)
    y, acc = ctx.gemm_i8(dev(qx), dev(qw), k, float(sx), dev(sw), q.ACT_NONE, want_y=True, want_acc=True)
    ctx.check_sync()
    ref = orc.int_gemm(qx[:, :k], qw[:, :k])
    np.testing.assert_array_equal(host(acc), ref)
    np.testing.assert_array_equal(host(y).view(np.uint32), orc.dequant_output(ref, sx, sw).view(np.uint32))


@pytest.mark.parametrize("m,n,k", [(5000, 1024, 272), (257, 300, 1040), (129, 2304, 64)])
def test_gemm_pair_and_single_cta_tiles_agree(ctx, m, n, k):
    """Outputs wider than 128 columns run on CTA pairs (256-row tiles); the single-CTA path must
    give the same bits, also when a pair works through several tiles and when the second CTA's
    rows or columns lie partly or wholly outside the matrix."""
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(m * 7 + n)
    ld = (k + 15) // 16 * 16
    qx, qw = _codes(rng, m, k, ld), _codes(rng, n, k, ld)
    sw = (10.0 ** rng.uniform(-4, -2, n)).astype(np.float32)
    res = []
    for pair in (True, False):
        ctx.set_pair_tiles(pair)
        try:
            y, acc = ctx.gemm_i8(dev(qx), dev(qw), k, 0.021, dev(sw), q.ACT_GELU_TANH, want_y=True, want_acc=True)
            ctx.check_sync()
        finally:
            ctx.set_pair_tiles(True)
        res.append((y, acc))
    np.testing.assert_array_equal(host(res[0][1]), orc.int_gemm(qx[:, :k], qw[:, :k]))
    assert torch.equal(res[0][1], res[1][1])
    assert torch.equal(res[0][0].view(torch.int32), res[1][0].view(torch.int32))


def test_gemm_i8_worst_case_magnitude(ctx):
    k = 4608
    qx = np.full((128, k), 127, np.int8)
    qw = np.full((32, k), -127, np.int8)
    qw[::2] = 127
    _, acc = ctx.gemm_i8(dev(qx), dev(qw), k, 1.0, None, want_y=False, want_acc=True)
    ctx.check_sync()
    np.testing.assert_array_equal(host(acc), orc.int_gemm(qx, qw))


@pytest.mark.parametrize("act", [1, 2])
def test_gemm_i8_activations(ctx, act):
    rng = np.random.default_rng(act)
    m, n, k = 513, 384, 256
    qx, qw = _codes(rng, m, k, k), _codes(rng, n, k, k)
    sw = (10.0 ** rng.uniform(-3.5, -2.5, n)).astype(np.float32)
    sx = np.float32(0.011)
    y, _ = ctx.gemm_i8(dev(qx), dev(qw), k, float(sx), dev(sw), act)
    ctx.check_sync()
    pre = orc.dequant_output(orc.int_gemm(qx, qw), sx, sw)
    ref = orc.activation(pre, act)
    if act == 1:
        np.testing.assert_array_equal(host(y), ref)
    else:
        assert np.abs(pre).max() > 3       # both tails are exercised
        np.testing.assert_allclose(host(y), ref, rtol=1e-6, atol=1e-6 * np.abs(ref).max())


@pytest.mark.parametrize("next_bits", [2, 4, 8, 16])
@pytest.mark.parametrize("m,n,k,act", [(300, 200, 150, 0), (1000, 768, 768, 1), (515, 1000, 256, 0), (260, 330, 144, 1)])
def test_gemm_i8_requant_codes_bit_exact(ctx, m, n, k, act, next_bits):
    rng = np.random.default_rng(m + n + k + next_bits)
    ld = (k + 15) // 16 * 16
    qx, qw = _codes(rng, m, k, ld), _codes(rng, n, k, ld)
    sw = (10.0 ** rng.uniform(-4, -2, n)).astype(np.float32)
    sx = np.float32(0.0173)
    y = orc.activation(orc.dequant_output(orc.int_gemm(qx[:, :k], qw[:, :k]), sx, sw), act)
    if next_bits == 16:
        out = ctx.gemm_i8_requant(dev(qx), dev(qw), k, float(sx), dev(sw), act, 1.0, 16)
        ctx.check_sync()
        got = host(out.float())[:, :n]
        np.testing.assert_array_equal(got.view(np.uint32), orc.bf16_round(y).view(np.uint32))
    else:
        A = np.float32(np.abs(y).max() * 0.6)            # calibrated maximum below the data: live clip
        _, inv = orc.scales_from_absmax(A, next_bits)
        out = ctx.gemm_i8_requant(dev(qx), dev(qw), k, float(sx), dev(sw), act, float(inv), next_bits)
        ctx.check_sync()
        want = orc.quantize(y, inv, next_bits)
        np.testing.assert_array_equal(host(out)[:, :n], want)
        assert np.abs(want).max() == orc.qmax(next_bits)


@pytest.mark.parametrize("m,n,k", [(64, 16, 16), (300, 200, 150), (1000, 768, 768), (129, 1000, 3072), (128, 1000, 2048)])
def test_gemm_bf16_matches_fp64_reference(ctx, m, n, k):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(m * n + k)
    x = rng.standard_normal((m, k)).astype(np.float32)
    w = (rng.standard_normal((n, k)) * 0.05).astype(np.float32)
    xq = ctx.quantize(dev(x), None, q.PER_TENSOR, 16)
    wq = ctx.quantize(dev(w), None, q.PER_TENSOR, 16)
    y = host(ctx.gemm_bf16(xq, wq, k))
    ctx.check_sync()
    ref = orc.bf16_gemm(x, w)
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) <= 1e-2
    assert np.abs(y - ref).max() <= 1e-2 * np.abs(ref).max()
    # fp32 accumulation of exact bf16 products: far tighter than the stated bound
    assert np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max() * np.sqrt(k)


# ----------------------------------------------------------------------------- host-side faults

def test_argument_errors_leave_outputs_untouched(ctx):
    import paper_2302_01382_b200 as q
    x = torch.ones((4, 32), device="cuda")
    with pytest.raises(q.QcfgError) as e:
        ctx.scales_from_absmax(x[0], 9)
    assert e.value.status == q.EBITS
    with pytest.raises(q.QcfgError) as e:
        ctx.quantize(x, x[0], q.PER_TENSOR, 12)
    assert e.value.status == q.EBITS
    with pytest.raises(q.QcfgError) as e:
        ctx.quantize(x, x[0], q.PER_TENSOR, 8, ldq=40)
    assert e.value.status == q.EALIGN
    with pytest.raises(q.QcfgError) as e:
        ctx.quant_error_sweep([x], b_lo=1, b_hi=8)
    assert e.value.status == q.EBITS
    qx = torch.zeros((8, 24), dtype=torch.int8, device="cuda")
    with pytest.raises(q.QcfgError) as e:
        ctx.gemm_i8(qx, qx, 24, 1.0, x[0])
    assert e.value.status == q.EALIGN
    assert "16-byte" in ctx.last_error()
    assert ctx.sync_status() == q.OK


# ----------------------------------------------------------------------------- device-side faults

def test_bounded_wait_gives_up_and_the_context_stays_usable(ctx):
    """Device waits on a barrier that is never signalled and on counters that never advance (the
    waits of the chained GEMM launches) each run into their limit (1 ms here); only when all of
    them gave up does the kernel report QCFG_ETIMEOUT through the error word.  The context is left
    able to run a correct GEMM."""
    import paper_2302_01382_b200 as q
    assert ctx.sync_status() == q.OK
    ctx.selftest_wait_timeout(1_000_000)
    assert ctx.sync_status() == q.ETIMEOUT
    assert "wait" in ctx.last_error()
    assert ctx.sync_status() == q.OK                  # the error word was cleared by the read
    rng = np.random.default_rng(5)
    qx = rng.integers(-127, 128, (200, 64), dtype=np.int8)
    qw = rng.integers(-127, 128, (48, 64), dtype=np.int8)
    _, acc = ctx.gemm_i8(dev(qx), dev(qw), 64, 1.0, None, want_y=False, want_acc=True)
    assert ctx.sync_status() == q.OK
    np.testing.assert_array_equal(host(acc), orc.int_gemm(qx, qw))
    with pytest.raises(q.QcfgError) as e:
        ctx.selftest_wait_timeout(0)
    assert e.value.status == q.EINVAL


def test_second_context_sweeps_wide_rows():
    """The sweep's shared-memory opt-in is set per context: a context created after another one
    has already swept still runs the variants that need more than 48 KB of shared memory."""
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(6)
    x = rng.standard_normal((40, 768)).astype(np.float32)
    so, ao = orc.quant_error_sweep([x])
    for _ in range(2):
        c = q.Context(0)
        sse, amax = c.quant_error_sweep([dev(x)])
        c.check_sync()
        np.testing.assert_allclose(host(sse), so, rtol=1e-5)
        np.testing.assert_array_equal(host(amax), ao)
        c.close()
