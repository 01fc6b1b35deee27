"""GPU parity of the BFP GEMMs through the C ABI: per-block integer sums bit-exact, outputs within
1e-6 of the FP32 accumulator magnitude of the oracle's order-free reference, and bit-equal to the
oracle's sequential accumulation where the kernel accumulates blocks in ascending order."""
import numpy as np
import pytest

import oracle
from paper_1804_01526_b200 import workloads as wl
from tests.helpers import gfmt, ofmt, to_dev

pytestmark = pytest.mark.gpu

TOL = 1e-6      # of the accumulator magnitude sum_kb |T|, as the target states


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


def run_spec(hb, sp, tensors, flags, expect_seq=True):
    A, B = tensors[sp.a_key], tensors[sp.b_key]
    ref = oracle.hbfp_gemm(sp.transA, sp.transB, A, B, ofmt(sp.fmt_a), ofmt(sp.fmt_b))
    C = hb.gemm(sp.transA, sp.transB, to_dev(A), to_dev(B), gfmt(sp.fmt_a), gfmt(sp.fmt_b), flags=flags)
    C = C.cpu().numpy()
    assert hb.device_status() == 0
    err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all(), (sp.name, float((err / np.maximum(ref["a_mag"], 1e-300)).max()))
    if expect_seq:
        assert np.array_equal(C, ref["c_seq"]), sp.name
    return C, ref


def impls(hb):
    return [hb.GEMM_FORCE_SIMT, hb.GEMM_AUTO]


@pytest.mark.parametrize("flag", ["simt", "auto"])
def test_single_256_cube(hb, flag):
    specs = wl.config_single_256()
    t = wl.materialize(specs, seed=0)
    run_spec(hb, specs[0], t, hb.GEMM_FORCE_SIMT if flag == "simt" else hb.GEMM_AUTO)


@pytest.mark.parametrize("flag", ["simt", "auto"])
def test_mlp_training_step_gemms(hb, flag):
    specs = wl.config_mlp()
    t = wl.materialize(specs, seed=1)
    for sp in specs:
        run_spec(hb, sp, t, hb.GEMM_FORCE_SIMT if flag == "simt" else hb.GEMM_AUTO,
                 expect_seq=(flag == "simt"))


@pytest.mark.parametrize("flag", ["simt", "auto"])
def test_resnet_im2col_gemms_reduced_batch(hb, flag):
    # batch 2 instead of 128 (M = 2048 / 512 rows): same K, N, formats and value laws
    specs = wl.config_resnet_im2col(batch=2)
    t = wl.materialize(specs, seed=2)
    for sp in specs:
        run_spec(hb, sp, t, hb.GEMM_FORCE_SIMT if flag == "simt" else hb.GEMM_AUTO,
                 expect_seq=(flag == "simt"))


@pytest.mark.parametrize("flag", ["simt", "auto"])
def test_transformer_gemms_reduced(hb, flag):
    # tokens 192, hidden 256: 12-bit hi/lo mantissas, 64 x 64 shared weight tiles, stochastic rounding
    specs = wl.config_transformer(tokens=192, hidden=256)
    t = wl.materialize(specs, seed=7)
    for sp in specs:
        run_spec(hb, sp, t, hb.GEMM_FORCE_SIMT if flag == "simt" else hb.GEMM_AUTO,
                 expect_seq=(flag == "simt"))


SMALL_CASES = [
    # transA, transB, M, N, K, mantissa bits, block, tile of B, rounding
    (0, 0, 128, 1024, 784, 8, 24, 24, 1),       # forward GEMM of the MLP configuration
    (0, 1, 128, 784, 1024, 8, 24, 24, 1),       # its backward-data GEMM (shared tiles read the other way)
    (1, 0, 784, 1024, 128, 8, 24, 0, 1),        # its backward-weight GEMM
    (0, 0, 1, 1, 1, 8, 32, 0, 0),
    (0, 0, 33, 95, 100, 6, 64, 0, 0),           # ragged in every dimension, two 32-byte steps per block
    (0, 0, 70, 50, 520, 8, 128, 0, 0),
    (1, 1, 40, 72, 900, 8, 200, 0, 1),          # blocks that span two 128-byte slices
    (0, 0, 64, 48, 300, 8, 0, 0, 0),            # one exponent per row / column
    (0, 0, 256, 256, 256, 4, 32, 32, 0),
]


@pytest.mark.parametrize("tA,tB,M,N,K,m,b,t,rounding", SMALL_CASES)
def test_small_problem_kernel_equals_the_sequential_definition(hb, tA, tB, M, N, K, m, b, t, rounding):
    """The tiled kernel for the smallest problems never splits K and adds blocks in ascending order: bit-equal to the oracle's c_seq."""
    A = wl.draw("lognormal", (K, M) if tA else (M, K), seed=31)
    B = wl.draw("he_weight", (N, K) if tB else (K, N), seed=32, fan_in=K)
    fa = dict(mant_bits=m, block=b, rounding=rounding, seed=4, stream_id=0)
    fb = dict(mant_bits=m, block=b, tile=t, rounding=rounding, seed=4, stream_id=1)
    ref = oracle.hbfp_gemm(tA, tB, A, B, ofmt(fa), ofmt(fb))
    C = hb.gemm(tA, tB, to_dev(A), to_dev(B), gfmt(fa), gfmt(fb), flags=hb.GEMM_FORCE_SMALL).cpu().numpy()
    assert hb.device_status() == 0 and hb.last_gemm_kernel() == "gemm_small_kernel"
    assert np.array_equal(C, ref["c_seq"])
    err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()


def test_small_problem_kernel_is_what_small_problems_get_and_large_ones_do_not(hb):
    fd = dict(mant_bits=8, block=64)
    A, B = wl.draw("normal", (256, 512), seed=33), wl.draw("normal", (512, 256), seed=34)
    hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd, stream_id=1))
    assert hb.last_gemm_kernel() == "gemm_small_kernel"
    A, B = wl.draw("normal", (1024, 2048), seed=35), wl.draw("normal", (2048, 1024), seed=36)
    hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd, stream_id=1))
    assert hb.last_gemm_kernel() == "gemm_tc_kernel"
    f12 = dict(mant_bits=12, block=64)
    with pytest.raises(hb.HbfpError) as e:
        hb.gemm(0, 0, to_dev(A[:64, :128].copy()), to_dev(B[:128, :64].copy()), gfmt(f12), gfmt(f12, stream_id=1), flags=hb.GEMM_FORCE_SMALL)
    assert e.value.code == hb.ERR_UNSUPPORTED


@pytest.mark.parametrize("impl", ["simt", "tensor"])
@pytest.mark.parametrize("m,b,M,N,K", [(8, 32, 200, 136, 288), (8, 128, 130, 260, 1024), (12, 64, 96, 72, 320),
                                       (8, 24, 50, 40, 100), (8, 0, 64, 64, 700), (8, 64, 128, 256, 512)])
def test_block_partials_are_bit_exact(hb, impl, m, b, M, N, K):
    A = wl.draw("lognormal", (M, K), seed=21)
    B = wl.draw("lognormal", (K, N), seed=22)
    fd = dict(mant_bits=m, block=b, rounding=1, seed=4)
    qA, sA = oracle.quantize(A, 1, ofmt(fd))
    qB, sB = oracle.quantize(B, 0, ofmt(fd, stream_id=1))
    ref = oracle.gemm(qA, sA, qB, sB, b, want_partials=True)
    pa = hb.quantize(to_dev(A), 1, gfmt(fd))
    pb = hb.quantize(to_dev(B), 0, gfmt(fd, stream_id=1))
    flag = hb.GEMM_FORCE_SIMT if impl == "simt" else hb.GEMM_FORCE_TENSOR
    try:
        P = hb.gemm_block_partials(pa, pb, flag)
    except hb.HbfpError as e:
        if impl == "tensor" and e.code == hb.ERR_UNSUPPORTED:
            pytest.skip("no tensor-core kernel for this case")
        raise
    assert np.array_equal(P.cpu().numpy(), ref["P"])
    assert hb.device_status() == 0


def test_backward_data_uses_packed_forward_weights(hb):
    """W is quantised ONCE into shared tiles; forward uses view c0 and backward-data view c1."""
    t, batch, fin, fout = 24, 64, 200, 136
    X = wl.draw("half_normal", (batch, fin), seed=31)
    W = wl.draw("he_weight", (fin, fout), seed=32, fan_in=fin)
    dY = wl.draw("grad", (batch, fout), seed=33)
    fw = dict(mant_bits=8, block=t, tile=t, rounding=1, seed=1, stream_id=1)
    fx = dict(mant_bits=8, block=t, rounding=1, seed=1, stream_id=0)
    fg = dict(mant_bits=8, block=t, rounding=1, seed=1, stream_id=2)
    c0, c1, _ = hb.quantize_tiles(to_dev(W), gfmt(fw))
    Y = hb.gemm_q(batch, fout, fin, to_dev(X), c0, transA=0, fmtA=gfmt(fx), flags=hb.GEMM_FORCE_SIMT).cpu().numpy()
    dX = hb.gemm_q(batch, fin, fout, to_dev(dY), c1, transA=0, fmtA=gfmt(fg), flags=hb.GEMM_FORCE_SIMT).cpu().numpy()
    assert np.array_equal(Y, oracle.hbfp_gemm(0, 0, X, W, ofmt(fx), ofmt(fw))["c_seq"])
    assert np.array_equal(dX, oracle.hbfp_gemm(0, 1, dY, W, ofmt(fg), ofmt(fw))["c_seq"])


def test_argument_errors_are_reported_not_thrown_by_cuda(hb):
    import torch
    A = torch.zeros((64, 64), device="cuda")
    f = hb.Format(8, 32)
    with pytest.raises(hb.HbfpError) as e:
        hb.gemm(0, 0, A, A, f, f, workspace=torch.empty(1024, dtype=torch.int8, device="cuda"))
    assert e.value.code == hb.ERR_WORKSPACE
    with pytest.raises(hb.HbfpError) as e:
        hb.gemm(0, 0, A, A, f, hb.Format(8, 64))
    assert e.value.code == hb.ERR_INVALID_ARG
    with pytest.raises(hb.HbfpError) as e:
        hb.quantize(A, 1, hb.Format(8, 32, rounding=5))
    assert e.value.code == hb.ERR_INVALID_ARG
    assert hb.device_status() == 0
    C = hb.gemm(0, 0, A[:0], A, f, f)          # empty M
    assert C.shape == (0, 64)


# The paired-SM kernel (two CTAs per 256 x 256 tile) needs at least 74 such tiles; these shapes span
# several tiles per SM pair, ragged edges in M, N and K, a second CTA whose half tile lies entirely
# outside the matrix (M % 256 <= 128, N % 256 <= 128), and all three blocks-per-stage variants.
PAIR_CASES = [
    # m, block, M, N, K
    (8, 128, 2560, 2048, 640),
    (8, 128, 2400, 2100, 1000),
    (8, 64, 2660, 2304, 448),
    (6, 64, 2304, 2188, 200),
    (8, 32, 2560, 2048, 288),
    (8, 100, 2688, 2176, 1000),
    (4, 16, 2330, 2332, 176),
]


@pytest.mark.parametrize("m,b,M,N,K", PAIR_CASES)
def test_paired_sm_kernel_matches_oracle_bit_for_bit(hb, m, b, M, N, K):
    A = wl.draw("lognormal", (M, K), seed=31)
    B = wl.draw("lognormal", (K, N), seed=32)
    fd = dict(mant_bits=m, block=b, rounding=0, seed=0)
    ref = oracle.hbfp_gemm(0, 0, A, B, ofmt(fd), ofmt(fd))
    C2 = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), flags=hb.GEMM_FORCE_TENSOR_2SM).cpu().numpy()
    assert hb.device_status() == 0
    err = np.abs(C2.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()
    assert np.array_equal(C2, ref["c_seq"])      # blocks accumulated in ascending order, no split-K
    C1 = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), flags=hb.GEMM_FORCE_TENSOR_1SM).cpu().numpy()
    assert np.array_equal(C1, C2)
    Ca = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), flags=hb.GEMM_AUTO).cpu().numpy()
    assert np.array_equal(Ca, C2)


def test_paired_sm_kernel_transposed_operands_and_stochastic_rounding(hb):
    # wgrad-shaped call: both operands are contracted along their row axis (column quantiser)
    M, N, K = 2304, 2304, 384
    X = wl.draw("half_normal", (K, M), seed=41)
    dY = wl.draw("grad", (K, N), seed=42)
    fa = dict(mant_bits=8, block=128, rounding=1, seed=9)
    ref = oracle.hbfp_gemm(1, 0, X, dY, ofmt(fa), ofmt(fa, stream_id=1))
    C = hb.gemm(1, 0, to_dev(X), to_dev(dY), gfmt(fa), gfmt(fa, stream_id=1), flags=hb.GEMM_FORCE_TENSOR_2SM).cpu().numpy()
    assert hb.device_status() == 0
    assert np.array_equal(C, ref["c_seq"])


def test_paired_sm_kernel_refuses_what_it_cannot_run(hb):
    A = to_dev(wl.draw("normal", (256, 256), seed=1))
    f8 = dict(mant_bits=8, block=128, rounding=0, seed=0)
    with pytest.raises(hb.HbfpError) as e:           # too few tiles to occupy the SM pairs
        hb.gemm(0, 0, A, A, gfmt(f8), gfmt(f8), flags=hb.GEMM_FORCE_TENSOR_2SM)
    assert e.value.code == hb.ERR_UNSUPPORTED
    big = to_dev(wl.draw("normal", (2560, 2048), seed=2))
    f12 = dict(mant_bits=12, block=64, rounding=0, seed=0)
    with pytest.raises(hb.HbfpError) as e:           # two mantissa planes
        hb.gemm(0, 1, big, big, gfmt(f12), gfmt(f12), flags=hb.GEMM_FORCE_TENSOR_2SM)
    assert e.value.code == hb.ERR_UNSUPPORTED


def test_mlp_step_captured_in_a_cuda_graph_replays_on_new_data(hb):
    """The calls are stream-ordered and allocate nothing when given their buffers, so a whole
    training step's GEMMs (stochastic rounding included: the draws depend on seed, stream id and
    element index only) can be captured once and replayed on new contents of the same tensors."""
    import torch
    specs = wl.config_mlp()
    t = wl.materialize(specs, seed=1)
    dev = {k: to_dev(v) for k, v in t.items()}
    outs = [torch.empty((sp.M, sp.N), dtype=torch.float32, device="cuda") for sp in specs]
    wss = [torch.empty(max(hb.gemm_workspace(sp.transA, sp.transB, sp.M, sp.N, sp.K, gfmt(sp.fmt_a), gfmt(sp.fmt_b)), 1),
                       dtype=torch.int8, device="cuda") for sp in specs]

    def step():
        for sp, C, ws in zip(specs, outs, wss):
            hb.gemm(sp.transA, sp.transB, dev[sp.a_key], dev[sp.b_key], gfmt(sp.fmt_a), gfmt(sp.fmt_b),
                    out=C, workspace=ws)

    step()                                   # eager: also sets the kernels' attributes once
    torch.cuda.synchronize()
    eager = [C.clone() for C in outs]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for C in outs:
        C.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert hb.device_status() == 0
    for sp, C, E in zip(specs, outs, eager):
        assert torch.equal(C, E), sp.name
    # new contents, same buffers: the replay must compute on them
    t2 = wl.materialize(specs, seed=5)
    for k, v in t2.items():
        dev[k].copy_(to_dev(v))
    graph.replay()
    torch.cuda.synchronize()
    assert hb.device_status() == 0
    for sp, C in zip(specs, outs):
        ref = oracle.hbfp_gemm(sp.transA, sp.transB, t2[sp.a_key], t2[sp.b_key], ofmt(sp.fmt_a), ofmt(sp.fmt_b))
        err = np.abs(C.cpu().numpy().astype(np.float64) - ref["c_ref"].astype(np.float64))
        assert (err <= TOL * ref["a_mag"]).all(), sp.name


@pytest.mark.parametrize("m,M,N,K", [(8, 128, 1024, 784), (8, 384, 512, 1024), (4, 200, 136, 1000), (12, 256, 256, 320)])
def test_one_exponent_per_row_no_blocks_no_tiles(hb, m, M, N, K):
    # "HBFP without tiles": block = 0, the whole contraction axis shares one exponent (one K-block per GEMM)
    A = wl.draw("half_normal", (M, K), seed=51)
    B = wl.draw("he_weight", (K, N), seed=52, fan_in=K)
    fd = dict(mant_bits=m, block=0, rounding=0, seed=0)
    ref = oracle.hbfp_gemm(0, 0, A, B, ofmt(fd), ofmt(fd))
    for flags in (hb.GEMM_FORCE_SIMT, hb.GEMM_AUTO):
        C = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), flags=flags).cpu().numpy()
        assert hb.device_status() == 0
        err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
        assert (err <= TOL * ref["a_mag"]).all()
        assert np.array_equal(C, ref["c_seq"])          # a single block: one product, one rounding


@pytest.mark.parametrize("M,N,K", [(128, 10, 1024), (1024, 10, 128), (200, 137, 256), (300, 66, 96)])
def test_tensor_core_kernel_writes_outputs_of_any_width(hb, M, N, K):
    # an output whose row pitch is not a multiple of four floats (the MLP's ten-class layer) cannot take
    # 16-byte stores; the tensor-core kernel then stores element by element
    A = wl.draw("half_normal", (M, K), seed=61)
    B = wl.draw("he_weight", (K, N), seed=62, fan_in=K)
    fd = dict(mant_bits=8, block=32, rounding=0, seed=0)
    ref = oracle.hbfp_gemm(0, 0, A, B, ofmt(fd), ofmt(fd))
    C = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), flags=hb.GEMM_FORCE_TENSOR).cpu().numpy()
    assert hb.device_status() == 0
    err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()
    # a view into a wider buffer with an odd pitch and an odd column offset
    import torch
    buf = torch.full((M, N + 7), -1.0, device="cuda")
    hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd), out=buf[:, 3:3 + N], flags=hb.GEMM_FORCE_TENSOR)
    out = buf.cpu().numpy()
    assert np.array_equal(out[:, 3:3 + N], C) and (out[:, :3] == -1).all() and (out[:, 3 + N:] == -1).all()


def _range_case(hb, A, B, flag):
    """GEMM of two FP32 matrices (8-bit mantissas, blocks of 128) on the kernel `flag` selects: returns
    (status return code, result, oracle reference)."""
    fd = dict(mant_bits=8, block=128)
    ref = oracle.hbfp_gemm(0, 0, A, B, ofmt(fd), ofmt(fd, stream_id=1))
    C = hb.gemm(0, 0, to_dev(A), to_dev(B), gfmt(fd), gfmt(fd, stream_id=1), flags=flag).cpu().numpy()
    rc, code = hb.device_status_rc()
    return rc, code, C, ref


@pytest.mark.parametrize("kernel", ["1sm", "2sm"])
def test_large_magnitudes_are_computed_or_reported_never_silently_wrong(hb, kernel):
    """Operands far from 1: the tensor-core kernels factor the block scale 2^(sA + sB); outside the
    range in which that is exact they must say so through the device status word."""
    flag = hb.GEMM_FORCE_TENSOR_1SM if kernel == "1sm" else hb.GEMM_FORCE_TENSOR_2SM
    M, N, K = 2304, 2304, 256            # 81 pair tiles: enough for the paired kernel
    rng = np.random.default_rng(77)
    B = wl.draw("normal", (K, N), seed=78)
    # (1) |A| ~ 2^60, |B| ~ 1: inside binary32, outside a fixed split of the scale
    A = (wl.draw("normal", (M, K), seed=79) * np.float32(2.0 ** 60)).astype(np.float32)
    rc, code, C, ref = _range_case(hb, A, B, flag)
    assert rc == hb.OK and code == 0
    assert np.array_equal(C, ref["c_seq"])
    # (2) |A| ~ 2^115: products are still finite with |B| ~ 2^-40
    A2 = (wl.draw("normal", (M, K), seed=80) * np.float32(2.0 ** 115)).astype(np.float32)
    B2 = (B * np.float32(2.0 ** -40)).astype(np.float32)
    rc, code, C, ref = _range_case(hb, A2, B2, flag)
    if rc == hb.OK:
        assert np.array_equal(C, ref["c_seq"])
    else:
        assert rc == hb.ERR_EXPONENT_RANGE and 900 <= code < 1000
    # (3) rows of one tile 140 binades apart: no split of the scale serves both
    A3 = wl.draw("normal", (M, K), seed=81)
    A3[0::2] *= np.float32(2.0 ** 70)
    A3[1::2] *= np.float32(2.0 ** -70)
    rc, code, C, ref = _range_case(hb, A3.astype(np.float32), B, flag)
    if rc == hb.OK:
        err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
        assert (err <= TOL * ref["a_mag"]).all()
    else:
        assert rc == hb.ERR_EXPONENT_RANGE and 900 <= code < 1000
    # the library is healthy afterwards
    rc, code, C, ref = _range_case(hb, wl.draw("normal", (M, K), seed=82), B, flag)
    assert rc == hb.OK and np.array_equal(C, ref["c_seq"])


def test_large_magnitudes_with_two_plane_mantissas_are_computed_or_reported(hb):
    """12-bit mantissas take the biased path of the single-SM kernel with a narrower exponent range
    (the bias is scaled by 256 * 2^sA): inside it the result is the oracle's, outside the status says so."""
    M, N, K = 384, 320, 256
    fd = dict(mant_bits=12, block=64)
    B = wl.draw("normal", (K, N), seed=178)
    for scale_a, scale_b in ((2.0 ** 60, 1.0), (2.0 ** 100, 2.0 ** -40), (2.0 ** 112, 2.0 ** -60), (1.0, 1.0)):
        A = (wl.draw("normal", (M, K), seed=179) * np.float32(scale_a)).astype(np.float32)
        Bs = (B * np.float32(scale_b)).astype(np.float32)
        ref = oracle.hbfp_gemm(0, 0, A, Bs, ofmt(fd), ofmt(fd, stream_id=1))
        C = hb.gemm(0, 0, to_dev(A), to_dev(Bs), gfmt(fd), gfmt(fd, stream_id=1), flags=hb.GEMM_FORCE_TENSOR_1SM).cpu().numpy()
        rc, code = hb.device_status_rc()
        if rc == hb.OK:
            assert np.array_equal(C, ref["c_seq"]), (scale_a, scale_b)
        else:
            assert scale_a > 2.0 ** 80 and rc == hb.ERR_EXPONENT_RANGE and 900 <= code < 1000
    assert rc == hb.OK            # the last, ordinary case ran clean


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_library_usable(hb):
    """The wait routine of the GEMM kernels, on a barrier nobody arrives on, with a budget of a few
    thousand cycles: the status word carries the code, the next read is clean, the next GEMM is right."""
    assert hb.device_status() == 0
    assert hb.selftest_bounded_wait(limit_cycles=5000, code=777) == 2      # abandoned, abort flag raised
    assert hb.device_status_rc() == (hb.ERR_TIMEOUT, 777)
    assert hb.device_status_rc() == (hb.OK, 0)
    specs = wl.config_single_256()
    run_spec(hb, specs[0], wl.materialize(specs, seed=0), hb.GEMM_AUTO)


def test_last_gemm_cycles_reports_the_paired_kernel_length(hb):
    """hbfp_last_gemm_cycles: the paired-SM kernel's length in SM cycles (longest CTA), a plausible number of them."""
    import torch
    n = 4096
    f = hb.Format(8, 128)
    A = to_dev(wl.draw("lognormal", (n, n), seed=71))
    pa, pb = hb.quantize(A, 1, f), hb.quantize(A, 0, f)
    ws = torch.empty(max(hb.gemm_q_workspace(n, n, n, pa, pb), 1), dtype=torch.int8, device="cuda")
    out = torch.empty((n, n), dtype=torch.float32, device="cuda")
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hb.gemm_q(n, n, n, pa, pb, out=out, workspace=ws, flags=hb.GEMM_FORCE_TENSOR_2SM)
    s.record()
    hb.gemm_q(n, n, n, pa, pb, out=out, workspace=ws, flags=hb.GEMM_FORCE_TENSOR_2SM)
    e.record()
    torch.cuda.synchronize()
    assert hb.last_gemm_kernel() == "gemm_tc2_kernel"
    cycles = hb.last_gemm_cycles()
    mhz = cycles / s.elapsed_time(e) / 1e3
    # 32 K-blocks x 4 tiles per cluster at several hundred cycles each; a clock between 0.5 and 2.2 GHz
    assert 32 * 4 * 300 < cycles < 32 * 4 * 20000
    assert 500 < mhz < 2200
    assert hb.device_status() == 0
