"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Tolerances: relative L2 <= 1e-3 (accuracy class TF32) /
1e-2 (class BF16) and max-abs <= 2e-2 * max|y_ref|; integer-valued cases bit-exact."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from oracle import winograd_exact as wx
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import assert_close, rel_l2, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available()
    B.lib()   # fails loudly if the extension is missing
    return torch


def run_layer(torch, layer, opts, inputs=None, check_status=True):
    x, w, b = inputs if inputs is not None else W.make_inputs(layer)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                          layer.dilation, opts)
    xd, wd, bd = to_dev(torch, x), to_dev(torch, w), to_dev(torch, b)
    y = r.run(xd, wd, bd)
    torch.cuda.synchronize()
    if check_status:
        assert r.device_status() == 0
    out = y.cpu().numpy()
    info = r.info
    r.close()
    return out, info, (x, w, b)


def oracle(layer, x, w, b):
    return oc.direct_conv(x, w, b, layer.stride, layer.pad, layer.dilation, layer.groups, layer.relu)


def opts_for(layer, **kw):
    return B.make_opts(groups=layer.groups, relu=layer.relu, **kw)


# ---------------------------------------------------------------------------
# Transforms and the checking contraction (no tensor cores): tight tolerances.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("m,k,pad,H,W_,Cin,Cout,N", [
    (2, 3, 1, 28, 28, 32, 32, 1), (4, 3, 1, 28, 28, 32, 32, 1), (6, 3, 1, 28, 28, 32, 32, 1),
    (4, 3, 1, 7, 7, 40, 24, 3), (6, 3, 1, 14, 14, 20, 50, 2), (2, 3, 0, 9, 11, 3, 5, 2),
    (2, 5, 2, 14, 14, 16, 16, 2), (4, 5, 2, 13, 10, 16, 16, 1), (2, 7, 3, 14, 14, 8, 8, 1),
    (4, 2, 0, 9, 9, 8, 8, 1), (2, 2, 1, 8, 8, 8, 8, 2), (6, 5, 2, 16, 16, 8, 8, 1), (4, 7, 3, 12, 12, 8, 8, 1)])
def test_winograd_fp32_reference_path(torch, m, k, pad, H, W_, Cin, Cout, N):
    layer = W.ConvLayer("t", N, Cin, Cout, H, W_, k, 1, pad, relu=True, x_dist="normal", w_dist="kaiming", seed=m * 100 + k)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=B.OPERAND_FP32_REF, passes=1)
    got, info, (x, w, b) = run_layer(torch, layer, o)
    assert info.algo == B.ALGO_WINOGRAD and info.m == m and info.alpha == m + k - 1
    ref = oracle(layer, x, w, b)
    e = rel_l2(got, ref)
    # fp32 transforms: error grows with alpha (larger matrix entries)
    assert e < (2e-5 if m + k - 1 <= 8 else 2e-3), e


@pytest.mark.parametrize("m,k,pid", [(2, 3, 2), (4, 3, 1), (6, 3, 3), (4, 5, 3)])
def test_input_and_weight_transform_stages(torch, m, k, pid):
    layer = W.ConvLayer("t", 2, 20, 24, 13, 11, k, 1, k // 2, relu=False, x_dist="normal", w_dist="normal", seed=77 + m)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=B.OPERAND_FP32_REF, passes=1, points_id=pid)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, k, 1, layer.pad, 1, o)
    info = r.info
    xd, wd = to_dev(torch, x), to_dev(torch, w)
    y = torch.zeros((layer.N, layer.Cout, info.OH, info.OW), device="cuda:0")
    r.run(xd, wd, None, y, stage_mask=B.STAGE_WEIGHT | B.STAGE_INPUT)
    torch.cuda.synchronize()
    a2 = info.alpha ** 2
    U = r.workspace_view(info.u_offset, a2 * layer.Cout * info.cin_pad * 4, torch.float32).cpu().numpy()
    U = U.reshape(a2, layer.Cout, info.cin_pad)
    V = r.workspace_view(info.v_offset, a2 * info.chunk_tiles * info.cin_pad * 4, torch.float32).cpu().numpy()
    V = V.reshape(a2, info.chunk_tiles, info.cin_pad)
    U_ref = wx.weight_transform_f64(w, m, pid)
    V_ref = wx.input_transform_f64(x, m, k, layer.pad, pid)
    assert V_ref.shape[1] == info.chunk_tiles
    assert rel_l2(U[:, :, :layer.Cin], U_ref) < 1e-6
    assert rel_l2(V[:, :, :layer.Cin], V_ref) < 1e-6
    # channel padding of both operands is zero
    assert not U[:, :, layer.Cin:].any() and not V[:, :, layer.Cin:].any()
    r.close()


@pytest.mark.parametrize("operand,passes,bits", [(B.OPERAND_TF32, 1, 10), (B.OPERAND_BF16, 1, 7)])
def test_operand_rounding_of_V(torch, operand, passes, bits):
    layer = W.ConvLayer("t", 1, 16, 16, 12, 12, 3, 1, 1, relu=False, x_dist="normal", w_dist="normal", seed=5)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=operand, passes=passes, points_id=1)
    r = B.ConvLayerRunner(1, 16, 16, 12, 12, 3, 1, 1, 1, o)
    info = r.info
    y = torch.zeros((1, 16, 12, 12), device="cuda:0")
    r.run(to_dev(torch, x), to_dev(torch, w), None, y, stage_mask=B.STAGE_INPUT)
    torch.cuda.synchronize()
    n = 36 * info.chunk_tiles * info.cin_pad
    if operand == B.OPERAND_TF32:
        V = r.workspace_view(info.v_offset, n * 4, torch.float32).cpu().numpy().astype(np.float64)
        # stored values carry at most 10 mantissa bits
        assert not (V.astype(np.float32).view(np.uint32) & 0x1FFF).any()
    else:
        V = r.workspace_view(info.v_offset, n * 2, torch.bfloat16).float().cpu().numpy().astype(np.float64)
    V = V.reshape(36, info.chunk_tiles, info.cin_pad)
    V_ref = wx.input_transform_f64(x, 4, 3, 1, 1)
    err = np.abs(V - V_ref)
    # within one unit in the last place of the operand format (fp32 evaluation + one rounding)
    assert (err <= np.abs(V_ref) * 2.0 ** (-bits) * 1.01 + 1e-6).all()
    r.close()


# ---------------------------------------------------------------------------
# The tensor-core contraction alone, on integer-valued operands: bit-exact.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("operand,passes", [(B.OPERAND_TF32, 1), (B.OPERAND_BF16, 1), (B.OPERAND_BF16, 3),
                                            (B.OPERAND_TF32, 3)])
@pytest.mark.parametrize("Cin,Cout,H", [(32, 32, 28), (72, 40, 13), (136, 272, 18)])
def test_contraction_bit_exact_on_integers(torch, operand, passes, Cin, Cout, H):
    m, k = 2, 3
    layer = W.ConvLayer("t", 2, Cin, Cout, H, H, k, 1, 1, relu=False, seed=9)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=operand, passes=passes, points_id=2)
    r = B.ConvLayerRunner(2, Cin, Cout, H, H, k, 1, 1, 1, o)
    info = r.info
    assert info.n_chunks == 1
    a2, T, Cp = 16, info.chunk_tiles, info.cin_pad
    rng = np.random.default_rng(Cin * 7 + Cout)
    U = rng.integers(-4, 5, (a2, Cout, Cp)).astype(np.float32)
    V = rng.integers(-4, 5, (a2, T, Cp)).astype(np.float32)
    U[:, :, Cin:] = 0
    tdt = torch.float32 if operand == B.OPERAND_TF32 else torch.bfloat16
    eb = 4 if operand == B.OPERAND_TF32 else 2
    split = 2 if passes == 3 else 1
    uview = r.workspace_view(info.u_offset, info.u_bytes, tdt)
    vview = r.workspace_view(info.v_offset, info.v_bytes, tdt)
    uview.zero_()
    vview.zero_()
    uview[:U.size] = to_dev(torch, U).to(tdt).flatten()
    vview[:V.size] = to_dev(torch, V).to(tdt).flatten()
    if split == 2:
        # a non-zero lo part: hi*hi + lo*hi + hi*lo must all arrive
        Ul = rng.integers(-2, 3, U.shape).astype(np.float32)
        Vl = rng.integers(-2, 3, V.shape).astype(np.float32)
        Ul[:, :, Cin:] = 0
        uview[info.u_bytes // 2 // eb: info.u_bytes // 2 // eb + U.size] = to_dev(torch, Ul).to(tdt).flatten()
        vview[info.v_bytes // 2 // eb: info.v_bytes // 2 // eb + V.size] = to_dev(torch, Vl).to(tdt).flatten()
    y = torch.zeros((2, Cout, info.OH, info.OW), device="cuda:0")
    r.run(None, None, None, y, stage_mask=B.STAGE_CONTRACT)
    torch.cuda.synchronize()
    assert r.device_status() == 0
    Mx = r.workspace_view(info.m_offset, a2 * Cout * info.m_row_stride * 4, torch.float32).cpu().numpy()
    Mx = Mx.reshape(a2, Cout, info.m_row_stride)[:, :, :T]
    ref = np.einsum("xoc,xtc->xot", U.astype(np.int64), V.astype(np.int64))
    if split == 2:
        ref = ref + np.einsum("xoc,xtc->xot", Ul.astype(np.int64), V.astype(np.int64)) \
                  + np.einsum("xoc,xtc->xot", U.astype(np.int64), Vl.astype(np.int64))
    assert np.array_equal(Mx.astype(np.int64), ref) and np.array_equal(Mx, ref.astype(np.float32))
    r.close()


# ---------------------------------------------------------------------------
# Whole path against the fp64 direct-convolution oracle.
# ---------------------------------------------------------------------------
def test_config0_both_tile_sizes(torch):
    layer = W.config0()[0]
    x, w, b = W.make_inputs(layer)
    ref = oracle(layer, x, w, b)
    seen = set()
    for m in (2, 4):
        o = opts_for(layer, precision=B.PREC_TF32, force_algo=B.ALGO_WINOGRAD, force_m=m)
        got, info, _ = run_layer(torch, layer, o, (x, w, b))
        assert info.algo == B.ALGO_WINOGRAD and info.m == m and info.operand != B.OPERAND_FP32_REF
        assert_close(got, ref, B.PREC_TF32, "config0 m=%d" % m)
        seen.add((info.operand, info.passes))
    assert seen


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("operand,passes,cls", [(B.OPERAND_TF32, 1, None), (B.OPERAND_BF16, 1, None),
                                                (B.OPERAND_TF32, 3, B.PREC_TF32), (B.OPERAND_BF16, 3, B.PREC_TF32)])
def test_forced_winograd_variants(torch, m, operand, passes, cls):
    """Every (m, operand, passes) runs; error stays within 2x of the planner's accuracy model, and
    within the class tolerance wherever the model admits the variant."""
    layer = W.ConvLayer("t", 2, 64, 48, 28, 28, 3, 1, 1, relu=True, seed=31)
    x, w, b = W.make_inputs(layer)
    ref = oracle(layer, x, w, b)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=operand, passes=passes)
    got, info, _ = run_layer(torch, layer, o, (x, w, b))
    e = rel_l2(got, ref)
    assert np.isfinite(got).all()
    assert e <= max(2.0 * info.predicted_error_ppm * 1e-6, 5e-6), (e, info.predicted_error_ppm)
    if cls is not None:
        assert_close(got, ref, cls, "m=%d" % m)


# Widths that are not a multiple of 4 (rows not 16-byte aligned) take the input transform that stages whole
# channel planes: planes up to 256 pixels and larger ones, channel counts below, off and above the 64-channel
# block, odd channel counts, non-square images, k = 5, and a plane too large for shared memory (33 x 33,
# which falls back to the ring kernel).  The integer run is bit-exact for F(2x2,3x3) with unit points, whose
# transforms are exact on small integers (entries 0, +-1, 1/2): every element of V was built from the right pixels.
@pytest.mark.parametrize("Cin,Cout,H,W_,k,m,N", [
    (3, 8, 14, 14, 3, 2, 2), (66, 24, 7, 7, 3, 4, 3), (130, 16, 13, 13, 3, 4, 1), (64, 32, 18, 18, 3, 6, 2),
    (17, 20, 17, 22, 3, 2, 1), (40, 8, 10, 30, 3, 4, 2), (24, 8, 30, 10, 3, 2, 1), (5, 4, 5, 6, 3, 2, 2),
    (32, 16, 15, 15, 5, 2, 1), (64, 16, 33, 33, 3, 4, 1)])
def test_winograd_on_planes_with_unaligned_rows(torch, Cin, Cout, H, W_, k, m, N):
    layer = W.ConvLayer("t", N, Cin, Cout, H, W_, k, 1, (k - 1) // 2, relu=True, seed=Cin + H + W_)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=B.OPERAND_BF16, passes=3)
    got, info, _ = run_layer(torch, layer, o, (x, w, b))
    assert info.algo == B.ALGO_WINOGRAD and info.m == m
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, "winograd, unaligned rows")
    if m == 2 and k == 3:
        xi, wi, bi = W.integer_inputs(layer, -2, 2)
        oi = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=2, operand=B.OPERAND_TF32, passes=1,
                      points_id=B.POINTS_UNIT)
        goti, _, _ = run_layer(torch, layer, oi, (xi, wi, bi))
        assert np.array_equal(goti.astype(np.float64), oracle(layer, xi, wi, bi))


@pytest.mark.parametrize("batch", [1, 3])
def test_config1_planner_choice(torch, batch):
    for layer in W.config1(1):
        layer = layer.with_batch(batch)
        x, w, b = W.make_inputs(layer)
        got, info, _ = run_layer(torch, layer, None, (x, w, b))       # mnn_conv_plan defaults
        assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, layer.name)


@pytest.mark.parametrize("cls", [B.PREC_TF32, B.PREC_BF16])
def test_config1_forced_winograd_by_class(torch, cls):
    for layer in W.config1(1):
        layer = layer.with_batch(2)
        x, w, b = W.make_inputs(layer)
        o = opts_for(layer, precision=cls, force_algo=B.ALGO_WINOGRAD)
        got, info, _ = run_layer(torch, layer, o, (x, w, b))
        assert info.algo == B.ALGO_WINOGRAD
        assert_close(got, oracle(layer, x, w, b), cls, layer.name)


def test_chunked_pipeline_matches_unchunked(torch):
    layer = W.ConvLayer("t", 5, 32, 32, 20, 20, 3, 1, 1, relu=True, seed=12)
    x, w, b = W.make_inputs(layer)
    ref = oracle(layer, x, w, b)
    outs = []
    for chunk in (5, 2, 1):
        o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_BF16, passes=3, chunk_images=chunk)
        got, info, _ = run_layer(torch, layer, o, (x, w, b))
        assert info.chunk_images == chunk and info.n_chunks == -(-5 // chunk)
        assert_close(got, ref, B.PREC_TF32, "chunk=%d" % chunk)
        outs.append(got)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_invariants_delta_zero_and_batch_permutation(torch):
    C, H = 16, 12
    layer = W.ConvLayer("t", 3, C, C, H, H, 3, 1, 1, relu=False, bias_dist="zero", x_dist="normal", seed=3)
    x, _, _ = W.make_inputs(layer)
    w = np.zeros((C, C, 3, 3), dtype=np.float32)
    for c in range(C):
        w[c, c, 1, 1] = 1.0
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_BF16, passes=3)
    got, _, _ = run_layer(torch, layer, o, (x, w, None))
    assert rel_l2(got, x) < 1e-4                      # delta kernel reproduces the input
    perm = [2, 0, 1]
    got_p, _, _ = run_layer(torch, layer, o, (x[perm], w, None))
    assert np.array_equal(got_p, got[perm])           # images are independent
    layer_b = W.ConvLayer("t", 1, C, C, H, H, 3, 1, 1, relu=True, seed=4)
    _, w2, b2 = W.make_inputs(layer_b)
    got_z, _, _ = run_layer(torch, layer_b, opts_for(layer_b, force_algo=B.ALGO_WINOGRAD, force_m=2),
                            (np.zeros((1, C, H, H), np.float32), w2, b2))
    expect = np.maximum(b2, 0)[None, :, None, None] * np.ones((1, C, H, H), np.float32)
    assert np.array_equal(got_z, expect.astype(np.float32))    # zero input -> ReLU(bias)


# ---------------------------------------------------------------------------
# GEMM and direct schemes.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("Cin,Cout,H,k,stride,pad,dil,N", [
    (64, 128, 14, 1, 1, 0, 1, 2), (64, 128, 28, 1, 2, 0, 1, 2), (32, 64, 15, 3, 2, 1, 1, 2),
    (24, 40, 17, 3, 1, 2, 2, 1), (3, 64, 32, 7, 2, 3, 1, 2), (100, 36, 9, 1, 1, 0, 1, 3), (16, 300, 10, 3, 1, 1, 1, 1),
    (3, 16, 150, 7, 2, 3, 1, 1), (80, 24, 20, 3, 2, 1, 1, 2), (6, 10, 9, 5, 1, 2, 1, 2), (8, 16, 33, 3, 1, 1, 3, 1),
    (4, 8, 5, 3, 1, 1, 1, 3), (2, 8, 12, 2, 2, 0, 1, 2), (40, 16, 70, 3, 1, 1, 1, 1)])
@pytest.mark.parametrize("operand", [B.OPERAND_TF32, B.OPERAND_BF16, B.OPERAND_FP32_REF])
def test_gemm_scheme(torch, Cin, Cout, H, k, stride, pad, dil, N, operand):
    layer = W.ConvLayer("t", N, Cin, Cout, H, H, k, stride, pad, dil, relu=True, seed=Cin + Cout)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_GEMM, operand=operand, precision=B.PREC_BF16 if operand == B.OPERAND_BF16 else 0)
    got, info, _ = run_layer(torch, layer, o, (x, w, b))
    assert info.algo == B.ALGO_GEMM
    ref = oracle(layer, x, w, b)
    if operand == B.OPERAND_FP32_REF:
        assert rel_l2(got, ref) < 1e-5
    else:
        assert_close(got, ref, B.PREC_BF16 if operand == B.OPERAND_BF16 else B.PREC_TF32, "gemm")


def test_gemm_bit_exact_on_integers(torch):
    layer = W.ConvLayer("t", 2, 24, 40, 11, 11, 3, 2, 1, relu=True, seed=1)
    x, w, b = W.integer_inputs(layer)
    ref = oracle(layer, x, w, b)
    for operand in (B.OPERAND_TF32, B.OPERAND_BF16):
        o = opts_for(layer, force_algo=B.ALGO_GEMM, operand=operand, precision=B.PREC_BF16)
        got, _, _ = run_layer(torch, layer, o, (x, w, b))
        assert np.array_equal(got.astype(np.float64), ref)


# 1x1 stride-1 layers: the GEMM scheme with either left operand (the gathered patch matrix, or x itself read as
# a pixel-contiguous operand).  Shapes cover one and several 32-pixel atoms per image with a ragged last atom,
# an atom count that does not fill the last work item, exactly four atoms, a last item of whole atoms only, a
# last item holding only the ragged atom, channel counts off the K block and the channel block.
@pytest.mark.parametrize("Cin,Cout,H,W_,N", [
    (64, 128, 8, 8, 2), (24, 40, 14, 14, 3), (512, 512, 14, 14, 1), (100, 72, 6, 6, 5), (32, 16, 28, 28, 2),
    (72, 300, 9, 12, 2), (130, 260, 7, 12, 7), (8, 8, 4, 8, 1), (16, 24, 8, 16, 2), (40, 48, 10, 16, 2),
    (33, 20, 16, 18, 1), (20, 24, 4, 9, 3),
    # images of more than four atoms: exactly eight atoms, seven and a ragged one, fifty atoms, two channel blocks
    (48, 64, 16, 16, 3), (16, 272, 12, 20, 2), (64, 96, 40, 40, 1), (96, 512, 14, 14, 4),
    # more work items than SMs (several items per CTA, both accumulator buffers in use): Cout 64 and 512, five
    # atoms, twenty-five atoms
    (32, 64, 14, 14, 80), (32, 512, 14, 14, 40), (16, 32, 10, 16, 80), (16, 16, 28, 28, 24)])
@pytest.mark.parametrize("lhs", [B.GEMM_LHS_PATCHES, B.GEMM_LHS_X])
def test_gemm_left_operand_1x1(torch, Cin, Cout, H, W_, N, lhs):
    layer = W.ConvLayer("t", N, Cin, Cout, H, W_, 1, 1, 0, 1, relu=True, seed=Cin + H)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_GEMM, operand=B.OPERAND_TF32, passes=1, gemm_lhs=lhs)
    got, info, _ = run_layer(torch, layer, o, (x, w, b))
    assert info.algo == B.ALGO_GEMM and info.gemm_lhs == lhs
    assert info.launches_per_run == (1 if lhs == B.GEMM_LHS_X else 2)
    if lhs == B.GEMM_LHS_X:
        assert info.v_bytes == 0
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, "gemm 1x1")


@pytest.mark.parametrize("Cin,Cout,H,N", [(40, 24, 6, 3), (96, 136, 14, 2)])
def test_gemm_left_operand_x_bit_exact_on_integers(torch, Cin, Cout, H, N):
    # small integers are exact in TF32 whether rounded or truncated: both left operands give the exact sums
    layer = W.ConvLayer("t", N, Cin, Cout, H, H, 1, 1, 0, 1, relu=False, seed=3)
    x, w, b = W.integer_inputs(layer)
    ref = oracle(layer, x, w, b)
    for lhs in (B.GEMM_LHS_PATCHES, B.GEMM_LHS_X):
        o = opts_for(layer, force_algo=B.ALGO_GEMM, operand=B.OPERAND_TF32, passes=1, gemm_lhs=lhs)
        got, info, _ = run_layer(torch, layer, o, (x, w, b))
        assert info.gemm_lhs == lhs
        assert np.array_equal(got.astype(np.float64), ref)


def test_gemm_left_operand_x_leaves_neighbours_untouched(torch):
    # the ragged last atom of an image must not write into the next channel's pixels: run into a buffer
    # prefilled with a marker and compare everything, then check two images give what each gives alone
    layer = W.ConvLayer("t", 2, 48, 20, 6, 6, 1, 1, 0, 1, relu=False, seed=11)
    x, w, b = W.make_inputs(layer)
    o = opts_for(layer, force_algo=B.ALGO_GEMM, operand=B.OPERAND_TF32, passes=1, gemm_lhs=B.GEMM_LHS_X)
    both, _, _ = run_layer(torch, layer, o, (x, w, b))
    one = W.ConvLayer("t", 1, 48, 20, 6, 6, 1, 1, 0, 1, relu=False, seed=11)
    for n in range(2):
        alone, _, _ = run_layer(torch, one, o, (x[n:n + 1].copy(), w, b))
        assert np.array_equal(alone[0], both[n])


@pytest.mark.parametrize("C,H,stride,N", [(32, 112, 1, 2), (64, 112, 2, 2), (40, 13, 1, 3), (40, 13, 2, 3), (8, 7, 1, 1),
                                          (8, 70, 2, 1), (16, 33, 1, 1)])
def test_depthwise_direct(torch, C, H, stride, N):
    layer = W.ConvLayer("t", N, C, C, H, H, 3, stride, 1, groups=C, relu=True, seed=C + H)
    x, w, b = W.make_inputs(layer)
    got, info, _ = run_layer(torch, layer, opts_for(layer), (x, w, b))
    assert info.algo == B.ALGO_DIRECT
    assert rel_l2(got, oracle(layer, x, w, b)) < 1e-6


# Even widths take the depthwise kernel with 2 or 4 columns per lane: widths that fill 8, 16 and 32 lanes, that
# need two and three overlapping strips, heights off the 32-row band and odd, plane counts that leave a warp
# partly empty, both strides.
@pytest.mark.parametrize("C,H,W_,N", [(10, 14, 14, 3), (7, 28, 28, 2), (6, 56, 56, 1), (3, 112, 112, 1), (2, 40, 224, 1),
                                      (3, 9, 130, 2), (5, 15, 6, 1), (4, 67, 36, 1), (1, 33, 248, 1), (9, 5, 2, 1),
                                      (2, 3, 500, 1)])
@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_even_widths(torch, C, H, W_, N, stride):
    layer = W.ConvLayer("t", N, C, C, H, W_, 3, stride, 1, groups=C, relu=(C % 2 == 0), seed=C + H + W_)
    x, w, b = W.make_inputs(layer)
    got, info, _ = run_layer(torch, layer, opts_for(layer), (x, w, b))
    assert info.algo == B.ALGO_DIRECT
    ref = oracle(layer, x, w, b)
    assert got.shape == ref.shape
    assert rel_l2(got, ref) < 1e-6
    # integer inputs: bit-exact, which also shows every output element was written exactly once with its own value
    xi, wi, bi = W.integer_inputs(layer)
    goti, _, _ = run_layer(torch, layer, opts_for(layer), (xi, wi, bi))
    assert np.array_equal(goti.astype(np.float64), oracle(layer, xi, wi, bi))


@pytest.mark.parametrize("Cin,Cout,H,k,stride,pad,dil,groups", [
    (3, 32, 32, 3, 2, 1, 1, 1), (3, 16, 30, 7, 2, 3, 1, 1), (6, 6, 9, 3, 1, 1, 2, 6), (5, 7, 8, 2, 1, 0, 1, 1),
    (4, 4, 6, 5, 3, 2, 1, 4), (16, 64, 11, 2, 1, 0, 2, 4), (32, 8, 14, 3, 2, 0, 1, 2), (8, 32, 13, 1, 1, 0, 1, 2),
    (64, 4, 9, 2, 2, 1, 2, 4), (3, 40, 37, 3, 2, 1, 1, 1), (3, 24, 19, 3, 1, 1, 1, 1), (3, 33, 50, 3, 2, 0, 1, 1)])
def test_generic_direct(torch, Cin, Cout, H, k, stride, pad, dil, groups):
    layer = W.ConvLayer("t", 2, Cin, Cout, H, H, k, stride, pad, dil, groups=groups, relu=True, seed=k)
    x, w, b = W.make_inputs(layer)
    got, info, _ = run_layer(torch, layer, opts_for(layer, force_algo=B.ALGO_DIRECT), (x, w, b))
    assert info.algo == B.ALGO_DIRECT
    assert rel_l2(got, oracle(layer, x, w, b)) < 1e-6


# Planes of at most 256 elements take the kernel that stages four whole planes per warp in shared memory: plane
# counts that leave the last group partial, odd and even widths (single outputs / output pairs), both strides,
# the smallest planes.
@pytest.mark.parametrize("C,H,W_,N", [(13, 14, 14, 5), (9, 7, 7, 7), (6, 16, 16, 2), (5, 3, 11, 3), (3, 1, 1, 2),
                                      (2, 2, 128, 1), (7, 15, 17, 1), (512, 14, 14, 2)])
@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_small_planes(torch, C, H, W_, N, stride):
    layer = W.ConvLayer("t", N, C, C, H, W_, 3, stride, 1, groups=C, relu=(C % 2 == 1), seed=C + H)
    x, w, b = W.make_inputs(layer)
    got, info, _ = run_layer(torch, layer, opts_for(layer), (x, w, b))
    assert info.algo == B.ALGO_DIRECT
    ref = oracle(layer, x, w, b)
    assert got.shape == ref.shape
    assert rel_l2(got, ref) < 1e-6
    xi, wi, bi = W.integer_inputs(layer)
    goti, _, _ = run_layer(torch, layer, opts_for(layer), (xi, wi, bi))
    assert np.array_equal(goti.astype(np.float64), oracle(layer, xi, wi, bi))


@pytest.mark.parametrize("Cout,H,Wd,relu", [(70, 30, 44, False), (32, 64, 64, True), (5, 2, 4, True), (21, 8, 12, False), (48, 100, 36, True)])
def test_stem_pixel_pairs(torch, Cout, H, Wd, relu):
    """3 -> Cout 3x3 stride 2 padding 1 with H even and W a multiple of 4: the kernel that owns two adjacent
    output pixels per thread; integers make the comparison exact, floats check the accumulation."""
    layer = W.ConvLayer("t", 3, 3, Cout, H, Wd, 3, 2, 1, 1, relu=relu, seed=Cout)
    x, w, b = W.make_inputs(layer)
    got, info, _ = run_layer(torch, layer, opts_for(layer, force_algo=B.ALGO_DIRECT), (x, w, b))
    assert info.algo == B.ALGO_DIRECT
    assert rel_l2(got, oracle(layer, x, w, b)) < 1e-6
    xi, wi, bi = W.integer_inputs(layer, -3, 3)
    goti, _, _ = run_layer(torch, layer, opts_for(layer, force_algo=B.ALGO_DIRECT), (xi, wi, bi))
    assert np.array_equal(goti.astype(np.float64), oracle(layer, xi, wi, bi))


def test_integer_direct_and_winograd_exact(torch):
    """Small integers: the direct kernel is exact; Winograd F(2,3) with unit points has
    transform entries that are multiples of 1/2 and 1/4, so it is exact too."""
    layer = W.ConvLayer("t", 2, 8, 8, 10, 10, 3, 1, 1, relu=False, seed=2)
    x, w, b = W.integer_inputs(layer, -2, 2)
    ref = oracle(layer, x, w, b)
    got, _, _ = run_layer(torch, layer, opts_for(layer, force_algo=B.ALGO_DIRECT), (x, w, b))
    assert np.array_equal(got.astype(np.float64), ref)
    o = opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=2, operand=B.OPERAND_TF32, passes=1, points_id=2)
    got, _, _ = run_layer(torch, layer, o, (x, w, b))
    assert np.array_equal(got.astype(np.float64), ref)


def test_error_paths(torch):
    layer = W.config0()[0]
    r = B.ConvLayerRunner(1, 32, 32, 28, 28, 3, 1, 1, 1, opts_for(layer, force_algo=B.ALGO_WINOGRAD, force_m=2))
    x = torch.zeros((1, 32, 28, 28), device="cuda:0")
    w = torch.zeros((32, 32, 3, 3), device="cuda:0")
    y = torch.zeros((1, 32, 28, 28), device="cuda:0")
    with pytest.raises(B.MnnError) as ei:
        B.mnn_conv_run(r.plan, x.data_ptr() + 4, w.data_ptr(), None, y.data_ptr(), r.stream())
    assert ei.value.code == B.MNN_EALIGN
    with pytest.raises(B.MnnError) as ei:
        B.mnn_conv_run(r.plan, x.data_ptr(), w.data_ptr(), None, x.data_ptr(), r.stream())
    assert ei.value.code == B.MNN_EINVAL
    with pytest.raises(B.MnnError) as ei:
        B.mnn_conv_set_workspace(r.plan, r._ws_ptr, 1024)
    assert ei.value.code == B.MNN_EWORKSPACE
    with pytest.raises(B.MnnError) as ei:          # the failed call dropped the workspace
        B.mnn_conv_run(r.plan, x.data_ptr(), w.data_ptr(), None, y.data_ptr(), r.stream())
    assert ei.value.code == B.MNN_EWORKSPACE
    r.close()
