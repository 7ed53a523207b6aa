"""Pins for the CPU oracle: closed forms, invariants, library routines on special cases, exact
brute force on tiny shapes.  CPU only.  A plausible mistake in the oracle (dropped term, wrong
sign or index, transposed operand, swapped op order) fails at least one test here."""
import math
import os
from dataclasses import replace

import mpmath as mp
import numpy as np
import pytest
import torch

from fc_inputs import rng, workloads as wl
from tests import brute

mp.mp.dps = 50
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, lo=-1.0, hi=1.0):
    return np.random.default_rng(seed).uniform(lo, hi, size=shape)


# ----------------------------------------------------------------------------- widening
def test_widen_bf16_all_patterns(orc):
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.widen(bits)
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    ok = (got == want) | (np.isnan(got) & np.isnan(want))
    assert ok.all()


def test_widen_f16_all_patterns(orc):
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.widen(bits.view(np.float16))
    want = torch.from_numpy(bits.view(np.int16)).view(torch.float16).to(torch.float64).numpy()
    ok = (got == want) | (np.isnan(got) & np.isnan(want))
    assert ok.all()
    assert orc.widen(np.array([1.0, -2.5, 65504.0, 2.0 ** -24], np.float16)).tolist() == [1.0, -2.5, 65504.0, 2.0 ** -24]


def test_widen_f32_exact(orc):
    a = np.array([0.1, -3.5, 1e-40, 3e38, -0.0], dtype=np.float32)
    assert np.array_equal(orc.widen(a), a.astype(np.float64))


# ----------------------------------------------------------------------------- GEMM NT
def test_gemm_identity_weight_returns_x(orc):
    X = _rand((7, 5), 1)
    assert np.array_equal(orc.gemm_nt(X, np.eye(5)), X)


def test_gemm_zero_weight_gives_bias_chain(orc):
    ch = wl.gemm_bias_relu_f32(6, 9, 5)
    X, W, b = wl.make_inputs(ch, 3)
    out = orc.run_chain(ch, [X, np.zeros_like(W), b])["main"]
    want = np.maximum(b.astype(np.float64), 0.0)
    assert np.array_equal(out, np.broadcast_to(want, (6, 9)))


def test_gemm_rank_one(orc):
    a = np.arange(1, 8, dtype=np.float64)          # M=7
    b = np.arange(-2, 3, dtype=np.float64)         # N=5
    K = 11
    A = np.repeat(a[:, None], K, 1)
    B = np.repeat(b[:, None], K, 1)
    assert np.array_equal(orc.gemm_nt(A, B), K * np.outer(a, b))


def test_gemm_one_hot_selects_entry(orc):
    # non-square everywhere: a transposed operand or swapped M/N index cannot pass
    M, N, K = 4, 6, 9
    A = np.zeros((M, K)); B = _rand((N, K), 2)
    A[2, 7] = 1.0
    V = orc.gemm_nt(A, B)
    assert np.array_equal(V[2], B[:, 7]) and np.count_nonzero(V[[0, 1, 3]]) == 0


def test_gemm_small_integers_exact(orc):
    r = np.random.default_rng(5)
    A = r.integers(-8, 9, size=(33, 70)).astype(np.float64)
    B = r.integers(-8, 9, size=(19, 70)).astype(np.float64)
    want = A.astype(np.int64) @ B.astype(np.int64).T
    assert np.array_equal(orc.gemm_nt(A, B), want.astype(np.float64))


def test_gemm_matches_library_matmul(orc):
    A = _rand((37, 129), 6); B = _rand((23, 129), 7)
    np.testing.assert_allclose(orc.gemm_nt(A, B), A @ B.T, rtol=0, atol=1e-12)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 2), (7, 5, 9)])
def test_gemm_chain_vs_exact_brute_force(orc, M, N, K):
    ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, variant="var")
    ins = wl.make_inputs(ch, 11)
    got = orc.run_chain(ch, ins)["main"]
    want = brute.run_chain(ch, ins)["main"]
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- conv
def _delta_weight(C, r, s):
    w = np.zeros((C, 3, 3, C))
    for c in range(C):
        w[c, r, s, c] = 1.0
    return w


def test_conv_centre_delta_is_identity(orc):
    x = _rand((2, 5, 7, 3), 8)
    assert np.array_equal(orc.conv2d_nhwc(x, _delta_weight(3, 1, 1), 1, 1), x)


def test_conv_shifted_delta_pins_direction_and_padding(orc):
    x = _rand((1, 5, 7, 2), 9)
    y = orc.conv2d_nhwc(x, _delta_weight(2, 0, 0), 1, 1)     # out[h][w] = in[h-1][w-1]
    assert np.array_equal(y[:, 1:, 1:, :], x[:, :-1, :-1, :])
    assert np.count_nonzero(y[:, 0, :, :]) == 0 and np.count_nonzero(y[:, :, 0, :]) == 0
    y2 = orc.conv2d_nhwc(x, _delta_weight(2, 2, 1), 1, 1)    # out[h][w] = in[h+1][w]
    assert np.array_equal(y2[:, :-1, :, :], x[:, 1:, :, :]) and np.count_nonzero(y2[:, -1]) == 0


def test_conv_all_ones_counts_valid_taps(orc):
    Cin, H, W = 4, 6, 5
    y = orc.conv2d_nhwc(np.ones((1, H, W, Cin)), np.ones((2, 3, 3, Cin)), 1, 1)
    assert y[0, 2, 2, 0] == 9 * Cin and y[0, 0, 2, 1] == 6 * Cin and y[0, 0, 0, 0] == 4 * Cin
    assert y[0, H - 1, W - 1, 1] == 4 * Cin
    pooled = orc.global_avgpool(y)
    want = Cin * (3 * H - 2) * (3 * W - 2) / (H * W)
    np.testing.assert_allclose(pooled, want, rtol=1e-15)


def test_pool_closed_form_at_benchmark_shape(orc):
    # all-ones 56x56x256 image and weights: mean over pixels of Cin * (#valid taps)
    H = W = 56
    taps = np.full((H, W), 9.0); taps[0, :] = taps[-1, :] = 6; taps[:, 0] = taps[:, -1] = 6
    taps[0, 0] = taps[0, -1] = taps[-1, 0] = taps[-1, -1] = 4
    V = (256.0 * taps)[None, :, :, None].repeat(3, axis=3)
    got = orc.global_avgpool(np.ascontiguousarray(V))
    assert got.shape == (1, 3)
    np.testing.assert_allclose(got, 256.0 * (3 * H - 2) * (3 * W - 2) / (H * W), rtol=1e-15)
    np.testing.assert_allclose(got, 2249.469387755102, rtol=1e-15)


@pytest.mark.parametrize("stride,pad,H,W", [(1, 1, 6, 5), (2, 1, 7, 8), (1, 0, 5, 5), (2, 0, 6, 9)])
def test_conv_matches_library_conv(orc, stride, pad, H, W):
    x = _rand((2, H, W, 3), 10); w = _rand((4, 3, 3, 3), 11)
    got = orc.conv2d_nhwc(x, w, stride, pad)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2),
                                     torch.from_numpy(w).permute(0, 3, 1, 2), stride=stride, padding=pad)
    np.testing.assert_allclose(got, ref.permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-13)


def test_conv_1x1_image_reduces_to_gemm(orc):
    x = _rand((5, 1, 1, 6), 12); w = _rand((4, 3, 3, 6), 13)
    got = orc.conv2d_nhwc(x, w, 1, 1).reshape(5, 4)
    want = orc.gemm_nt(np.ascontiguousarray(x.reshape(5, 6)), np.ascontiguousarray(w[:, 1, 1, :]))
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-15)


def test_conv_chain_vs_exact_brute_force(orc):
    ch = wl.conv_bias_relu_avgpool(batch=2, H=4, W=3, Cin=3, Cout=2)
    ins = wl.make_inputs(ch, 4)
    got = orc.run_chain(ch, ins)
    want = brute.run_chain(ch, ins)
    np.testing.assert_allclose(got["main"], want["main"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(got["reduce"], want["reduce"], rtol=0, atol=1e-14)


@pytest.mark.parametrize("stride,pad,H,W", [(1, 1, 6, 5), (2, 1, 7, 8), (1, 0, 5, 5), (2, 2, 6, 9)])
def test_conv_nchw_matches_library_conv(orc, stride, pad, H, W):
    """Channel-first storage: the library's convolution takes exactly these layouts, no permutation of the
    inputs; only the result is moved to channels-last."""
    x = _rand((2, 3, H, W), 14); w = _rand((4, 3, 3, 2), 15)
    got = orc.conv2d_nchw(x, w, stride, pad)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), stride=stride, padding=pad)
    np.testing.assert_allclose(got, ref.permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-13)


def test_conv_nchw_deltas_and_tap_counts(orc):
    """A delta at (r, s) = (0, 2) in channel c -> c + 1 (cyclic): out[h][w][c+1] = in[c][h-1][w+1], zeros where the
    tap leaves the image: pins the order of all four weight axes and of the image axes.  All-ones: valid taps."""
    C, H, W = 3, 5, 7
    x = _rand((2, C, H, W), 16)
    w = np.zeros((C, C, 3, 3))
    for c in range(C):
        w[(c + 1) % C, c, 0, 2] = 1.0
    y = orc.conv2d_nchw(x, w, 1, 1)
    for c in range(C):
        assert np.array_equal(y[:, 1:, :-1, (c + 1) % C], x[:, c, :-1, 1:])
    assert np.count_nonzero(y[:, 0, :, :]) == 0 and np.count_nonzero(y[:, :, -1, :]) == 0
    ones = orc.conv2d_nchw(np.ones((1, 4, 6, 5)), np.ones((2, 4, 3, 3)), 1, 1)
    assert ones[0, 2, 2, 0] == 36 and ones[0, 0, 2, 1] == 24 and ones[0, 0, 0, 0] == 16 and ones[0, 5, 4, 1] == 16


def test_conv_nchw_equals_nhwc_on_permuted_arrays(orc):
    x = _rand((2, 5, 6, 7), 17); w = _rand((3, 5, 2, 3), 18)       # non-square filter, stride 2
    a = orc.conv2d_nchw(x, w, 2, 1)
    b = orc.conv2d_nhwc(np.ascontiguousarray(x.transpose(0, 2, 3, 1)), np.ascontiguousarray(w.transpose(0, 2, 3, 1)), 2, 1)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-14)


def test_conv_nchw_chain_vs_exact_brute_force(orc):
    ch = wl.conv_nchw(wl.conv_bias_relu_avgpool(batch=2, H=4, W=5, Cin=3, Cout=2, R=3, S=3, pad=1))
    ins = wl.make_inputs(ch, 5)
    assert ins[0].shape == (2, 3, 4, 5) and ins[1].shape == (2, 3, 3, 3)
    got = orc.run_chain(ch, ins)
    want = brute.run_chain(ch, ins)
    np.testing.assert_allclose(got["main"], want["main"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(got["reduce"], want["reduce"], rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- elementwise ops
def test_relu_scale_clamp_exhaustive_bf16(orc):
    bits = np.arange(65536, dtype=np.uint16)
    v = orc.widen(bits)
    v = v[np.isfinite(v)]
    a = v.copy(); orc.apply_op(a, ("relu",), [])
    assert np.array_equal(a, np.where(v < 0, 0.0, v))
    a = v.copy(); orc.apply_op(a, ("scale", 0.5), [])
    assert np.array_equal(a, v * 0.5)
    a = v.copy(); orc.apply_op(a, ("clamp", -1.0, 1.0), [])
    assert np.array_equal(a, np.clip(v, -1.0, 1.0))
    assert a.max() == 1.0 and a.min() == -1.0


def test_bias_affine_add_broadcast_axis(orc):
    V = _rand((3, 4), 14); g = np.array([1., 2., 3., 4.]); b = np.array([10., 20., 30., 40.])
    a = V.copy(); orc.apply_op(a, ("bias_n", 0), [b]); assert np.array_equal(a, V + b[None, :])
    a = V.copy(); orc.apply_op(a, ("affine_n", 0, 1), [g, b]); assert np.array_equal(a, V * g[None, :] + b[None, :])
    T = _rand((3, 4), 15)
    a = V.copy(); orc.apply_op(a, ("add_tensor", 0), [T]); assert np.array_equal(a, V + T)


def test_gelu_tanh_values_and_identities(orc):
    pts = np.array([-6.0, -3.0, -2.0, -1.0, -0.5, -1e-3, 0.0, 1e-3, 0.5, 1.0, 2.0, 3.0, 6.0, 11.0])
    g = pts.copy(); orc.apply_op(g, ("gelu_tanh",), [])
    want = np.array([float(brute.gelu_tanh(mp.mpf(float(v)))) for v in pts])
    # 1 + tanh(.) cancels near v = -6 in fp64: absolute error there is ~1e-17 * |v|
    np.testing.assert_allclose(g, want, rtol=1e-14, atol=1e-15)
    assert g[6] == 0.0
    # G(v) - G(-v) = v because tanh is odd
    sym = np.array([0.3, 1.0, 2.5, 4.0]); gp = sym.copy(); gm = -sym
    orc.apply_op(gp, ("gelu_tanh",), []); orc.apply_op(gm, ("gelu_tanh",), [])
    np.testing.assert_allclose(gp - gm, sym, rtol=1e-14)
    # limits and a library routine
    assert abs(g[-1] - 11.0) < 1e-12 and abs(g[0]) < 1e-9
    v = _rand((1000,), 16, -5, 5)
    a = v.copy(); orc.apply_op(a, ("gelu_tanh",), [])
    ref = torch.nn.functional.gelu(torch.from_numpy(v), approximate="tanh").numpy()
    np.testing.assert_allclose(a, ref, rtol=0, atol=1e-14)


def test_op_order_is_respected(orc):
    # clamp(scale(v)) differs from scale(clamp(v)); relu(bias) differs from bias(relu)
    v = np.array([[3.0, -3.0]])
    a = v.copy(); orc.apply_op(a, ("scale", 0.5), []); orc.apply_op(a, ("clamp", -1.0, 1.0), [])
    assert np.array_equal(a, [[1.0, -1.0]])
    ch = replace(wl.gemm_bias_relu_f32(1, 2, 1), ops=(("relu",), ("bias_n", 2)))
    out = orc.run_chain(ch, [np.array([[1.0]], np.float32), np.array([[-2.0], [2.0]], np.float32),
                             np.array([-1.0, -1.0], np.float32)])["main"]
    assert np.array_equal(out, [[-1.0, 1.0]])


# ----------------------------------------------------------------------------- reductions
def test_lse_size_one_is_identity_golden(orc):
    vals = [float(l) for l in open(os.path.join(GOLDEN, "lse_size_one.txt")) if l.strip() and not l.startswith("#")]
    V = np.array(vals).reshape(-1, 1)
    assert np.array_equal(orc.row_logsumexp(V), np.array(vals))


def test_lse_closed_forms(orc):
    N = 4096
    out = orc.row_logsumexp(np.full((2, N), 2.5))
    np.testing.assert_allclose(out, 2.5 + 8.317766166719343, rtol=1e-15)
    v = _rand((5, 300), 17, -4, 4)
    base = orc.row_logsumexp(v)
    for c in (1e4, -1e4, 3.0):
        np.testing.assert_allclose(orc.row_logsumexp(v + c), base + c, rtol=1e-13)
    assert np.all(base >= v.max(1)) and np.all(base <= v.max(1) + math.log(300))
    dom = np.full((1, 50), -800.0); dom[0, 17] = 42.0
    assert orc.row_logsumexp(dom)[0] == 42.0
    want = [float(mp.log(mp.fsum([mp.exp(mp.mpf(float(x))) for x in row]))) for row in v]
    np.testing.assert_allclose(base, want, rtol=1e-14)
    np.testing.assert_allclose(base, torch.logsumexp(torch.from_numpy(v), 1).numpy(), rtol=1e-14)


def test_softmax_properties(orc):
    v = _rand((6, 257), 18, -6, 6)
    P = orc.row_softmax(v)
    assert np.abs(P.sum(1) - 1).max() <= 1e-12
    np.testing.assert_allclose(orc.row_softmax(v + 1234.5), P, rtol=1e-11)
    np.testing.assert_allclose(orc.row_softmax(np.full((1, 64), -3.0)), 1 / 64, rtol=1e-15)
    np.testing.assert_allclose(np.log(P), v - orc.row_logsumexp(v)[:, None], rtol=0, atol=1e-12)
    order = np.argsort(v[0]); assert np.all(np.diff(P[0][order]) >= 0)
    np.testing.assert_allclose(P, torch.softmax(torch.from_numpy(v), 1).numpy(), rtol=1e-13)


def test_row_sum_max_mean(orc):
    V = _rand((5, 37), 23, -3, 3)
    np.testing.assert_allclose(orc.row_sum(V), V.sum(1), rtol=0, atol=1e-13)
    assert np.array_equal(orc.row_max(V), V.max(1))
    ints = np.arange(1.0, 101.0)[None, :].repeat(2, 0)
    assert np.array_equal(orc.row_sum(np.ascontiguousarray(ints)), [5050.0, 5050.0])
    one = np.full((1, 9), -7.5); one[0, 4] = 2.0
    assert orc.row_max(one)[0] == 2.0 and orc.row_sum(one)[0] == -58.0
    from dataclasses import replace as _r
    for red in ("row_sum", "row_max", "row_mean"):
        ch = _r(wl.affine_gelu_residual_lse(3, 9), reduce=red)
        ins = wl.make_inputs(ch, 5)
        got, want = orc.run_chain(ch, ins), brute.run_chain(ch, ins)
        np.testing.assert_allclose(got["reduce"], want["reduce"], rtol=1e-13, atol=1e-14)
    ch = _r(wl.affine_gelu_residual_lse(4, 16), reduce="row_mean", ops=())
    x = wl.make_inputs(ch, 1)[0]
    np.testing.assert_allclose(orc.run_chain(ch, [x])["reduce"], rng.bf16_bits_to_f32(x).astype(np.float64).mean(1), atol=1e-15)


def test_avgpool_properties(orc):
    V = _rand((2, 3, 4, 5), 19); U = _rand((2, 3, 4, 5), 20)
    np.testing.assert_allclose(orc.global_avgpool(np.full((2, 3, 4, 5), 7.25)), 7.25, rtol=1e-15)
    np.testing.assert_allclose(orc.global_avgpool(2 * V + U), 2 * orc.global_avgpool(V) + orc.global_avgpool(U), atol=1e-15)
    np.testing.assert_allclose(orc.global_avgpool(V), V.mean(axis=(1, 2)), atol=1e-15)
    # pixel/channel index not swapped: one hot pixel in one channel
    Z = np.zeros((1, 3, 4, 5)); Z[0, 2, 1, 3] = 12.0
    want = np.zeros((1, 5)); want[0, 3] = 1.0
    assert np.array_equal(orc.global_avgpool(Z), want)


# ----------------------------------------------------------------------------- whole chains
def test_all_five_patterns_vs_brute_force(orc):
    chains = [wl.gemm_bias_relu_f32(3, 5, 7, variant="var"),
              wl.affine_gelu_residual_lse(3, 9),
              wl.gemm_bias_gelu_scale_clamp(5, 3, 4, variant="var"),
              wl.gemm_softmax(3, 7, 5, variant="var"),
              wl.conv_bias_relu_avgpool(batch=1, H=3, W=3, Cin=2, Cout=3)]
    for ch in chains:
        ins = wl.make_inputs(ch, 21)
        got, want = orc.run_chain(ch, ins), brute.run_chain(ch, ins)
        for k in want:
            np.testing.assert_allclose(got[k], want[k], rtol=1e-13, atol=1e-14, err_msg=f"{ch.name}:{k}")


def test_elementwise_chain_matches_library_sequence(orc):
    ch = wl.affine_gelu_residual_lse(17, 130)
    ins = wl.make_inputs(ch, 22)
    x, g, b, r = [torch.from_numpy(rng.bf16_bits_to_f32(a)).double() for a in ins]
    y = torch.nn.functional.gelu(x * g + b, approximate="tanh") + r
    got = orc.run_chain(ch, ins)
    np.testing.assert_allclose(got["main"], y.numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(got["reduce"], torch.logsumexp(y, 1).numpy(), rtol=1e-13)


def test_maxpool_2x2_against_reshape_and_planted_maxima(orc):
    """Non-overlapping 2x2 windows: numpy's reshape-and-max on even sizes; one planted maximum per
    window recovered at the right output position; an odd last row / column belongs to no window."""
    r = np.random.default_rng(5)
    V = r.standard_normal((3, 6, 8, 5))
    want = V.reshape(3, 3, 2, 4, 2, 5).max(axis=(2, 4))
    assert np.array_equal(orc.maxpool_2x2(V), want)
    # planted: window (i, j) of image b, channel c holds the value 100 + its own index at a random corner
    Z = -np.abs(r.standard_normal((2, 4, 6, 3)))
    tag = np.zeros((2, 2, 3, 3))
    for b in range(2):
        for i in range(2):
            for j in range(3):
                for c in range(3):
                    di, dj = r.integers(0, 2, 2)
                    tag[b, i, j, c] = 100 + ((b * 2 + i) * 3 + j) * 3 + c
                    Z[b, 2 * i + di, 2 * j + dj, c] = tag[b, i, j, c]
    assert np.array_equal(orc.maxpool_2x2(Z), tag)
    # odd sizes: the last row and column are dropped, so poisoning them changes nothing
    W = r.standard_normal((1, 5, 7, 2))
    base = orc.maxpool_2x2(W)
    assert base.shape == (1, 2, 3, 2)
    W2 = W.copy(); W2[:, 4, :, :] = 1e9; W2[:, :, 6, :] = 1e9
    assert np.array_equal(orc.maxpool_2x2(W2), base)
    assert np.array_equal(base, W[:, :4, :6].reshape(1, 2, 2, 3, 2, 2).max(axis=(2, 4)))
    # max commutes with a monotone map: pooling ReLU(V) equals ReLU of pooled V
    assert np.array_equal(orc.maxpool_2x2(np.maximum(V, 0)), np.maximum(orc.maxpool_2x2(V), 0))


# ----------------------------------------------------------------------------- 16-bit rounding and chained linear layers
def test_round_to_16_bit_grids(orc):
    """Rounding onto the bf16 / fp16 grids: every stored pattern is a fixed point; numpy's and the input
    generator's own conversions agree on random values; exact ties go to the even neighbour; an exact
    rational restatement agrees on values with long fractions."""
    pats = np.arange(65536, dtype=np.uint16)
    w = orc.widen(pats)
    fin = np.isfinite(w)
    assert np.array_equal(orc.round_to(w[fin], "bf16"), w[fin])
    h = pats.view(np.float16).astype(np.float64)
    finh = np.isfinite(h)
    assert np.array_equal(orc.round_to(h[finh], "f16"), h[finh])
    r = np.random.default_rng(11)
    x = (r.standard_normal(200000) * np.exp(r.uniform(-30, 30, 200000))).astype(np.float32)
    want_bf16 = rng.bf16_bits_to_f32(rng.f32_to_bf16_bits(x)).astype(np.float64)       # integer bit arithmetic
    assert np.array_equal(orc.round_to(x.astype(np.float64), "bf16"), want_bf16)
    xs = (r.standard_normal(200000) * np.exp(r.uniform(-12, 10, 200000))).astype(np.float32)
    with np.errstate(over="ignore"):
        want_f16 = xs.astype(np.float16).astype(np.float64)                              # numpy's conversion
    assert np.array_equal(orc.round_to(xs.astype(np.float64), "f16"), want_f16)
    # ties: 1 + 2^-8 lies halfway between bf16 neighbours 1 and 1 + 2^-7 -> 1 (even); 1 + 3*2^-8 -> 1 + 2^-6
    assert orc.round_to(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8)]), "bf16").tolist() == [1.0, 1 + 2.0 ** -6, -1.0]
    assert orc.round_to(np.array([1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11]), "f16").tolist() == [1.0, 1 + 2.0 ** -9]
    # just above a tie rounds up (a double rounding through fp32 would get this wrong)
    assert orc.round_to(np.array([1 + 2.0 ** -8 + 2.0 ** -40]), "bf16")[0] == 1 + 2.0 ** -7
    # subnormal and overflow ends of the fp16 grid
    assert orc.round_to(np.array([2.0 ** -25, 3 * 2.0 ** -25, 65519.9, 65520.0]), "f16").tolist() == [0.0, 2.0 ** -23, 65504.0, np.inf]
    from fractions import Fraction
    for v in [0.3, -7.123456789, 1e-3, 255.5, 3.0e5]:
        assert Fraction(float(orc.round_to(np.array([v]), "bf16")[0])) == brute.round_to_grid_fraction(Fraction(v), 8, -133)
        if abs(v) < 65504:
            assert Fraction(float(orc.round_to(np.array([v]), "f16")[0])) == brute.round_to_grid_fraction(Fraction(v), 11, -24)


def test_chained_linear_layers(orc):
    """x -> relu(x W1^T + b1) -> round to bf16 -> . W2^T + b2: identity second layer returns the rounded
    activations; exact-rational brute force (different loop order, rational rounding) agrees to 1e-12."""
    ch = wl.mlp(5, (16, 8, 8))
    ins = wl.make_inputs(ch, 2)
    ins[3] = rng.store(np.eye(8, dtype=np.float32), "bf16")
    ins[4] = rng.store(np.zeros(8, np.float32), "bf16")
    x = [orc.widen(a) for a in ins]
    h = np.maximum(orc.gemm_nt(x[0], x[1]) + x[2], 0.0)
    assert np.array_equal(orc.run_chain(ch, ins)["main"], orc.round_to(h, "bf16"))
    from fractions import Fraction
    ch = wl.mlp(3, (8, 8, 16, 8))
    ins = wl.make_inputs(ch, 4)
    got = orc.run_chain(ch, ins)["main"]
    f = [brute.to_fraction_array(a) for a in ins]
    v = brute.gemm_nt(f[0], f[1])
    for l, (wi, bi) in enumerate([(1, 2), (3, 4), (5, 6)]):
        if l > 0:
            v = np.vectorize(lambda t: brute.round_to_grid_fraction(t, 8, -133), otypes=[object])(v)
            v = brute.gemm_nt(v, f[wi])
        v = v + f[bi][None, :]
        if l < 2:
            v = np.vectorize(lambda t: t if t > 0 else Fraction(0), otypes=[object])(v)
    want = np.array([[float(t) for t in row] for row in v])
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    assert got.shape == (3, 8)


def test_widen_f8e4m3_all_patterns_and_generator_rounding(orc):
    """All 256 E4M3 patterns against the library's own conversion (torch float8_e4m3fn), the closed form of a
    few patterns, and the input generator's rounding against the library's on random values."""
    pats = np.arange(256, dtype=np.uint8)
    got = orc.widen(pats)
    want = torch.from_numpy(pats).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.isnan(got).sum() == 2
    assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    assert got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0x38] == 1.0 and got[0x7E] == 448.0 and got[0xB8] == -1.0
    r = np.random.default_rng(3)
    x = np.clip(r.standard_normal(50000) * np.exp(r.uniform(-8, 5, 50000)), -440, 440).astype(np.float32)
    assert np.array_equal(rng.f32_to_e4m3_bits(x), torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy())
    assert rng.f32_to_e4m3_bits(np.array([2.0 ** -10, 3 * 2.0 ** -10, 1e4, -1e4], np.float32)).tolist() == [0, 2, 0x7E, 0xFE]


def test_f8_gemm_chain_small_integers_and_brute_force(orc):
    ch = wl.gemm_f8_bias_gelu_scale_clamp(4, 5, 16, out_dtype="f32")
    ins = wl.make_inputs(ch, 1)
    got = orc.run_chain(replace(ch, ops=()), ins)["main"]
    a, b = orc.widen(ins[0]), orc.widen(ins[1])
    np.testing.assert_allclose(got, a @ b.T, rtol=0, atol=1e-12)      # library matmul on the widened operands
    from fractions import Fraction
    fa = np.array([[Fraction(float(v)) for v in row] for row in a], dtype=object)
    fb = np.array([[Fraction(float(v)) for v in row] for row in b], dtype=object)
    exact = brute.gemm_nt(fa, fb)
    assert all(Fraction(float(got[i, j])) == exact[i, j] for i in range(4) for j in range(5))   # 4-bit significands: exact in fp64


# ------------------------------------------------------------------ block-scaled (MX) contraction
def test_widen_e8m0_all_patterns(orc):
    """All 256 scale bytes against the library's own E8M0 type and the format's corner values: 127 is one, 0 the
    smallest scale 2^-127, 254 the largest 2^127, 255 not a number; neighbouring bytes differ by a factor of two."""
    pats = np.arange(256, dtype=np.uint8)
    got = orc.widen(pats.view(np.int8))
    want = torch.from_numpy(pats).view(torch.float8_e8m0fnu).to(torch.float64).numpy()
    assert np.array_equal(got[:255], want[:255]) and np.isnan(got[255]) and np.isnan(want[255])
    assert got[127] == 1.0 and got[0] == 2.0 ** -127 and got[254] == 2.0 ** 127
    assert np.array_equal(got[1:255] / got[0:254], np.full(254, 2.0))
    # the generator stores exponent x as byte x + 127 and keeps to the finite patterns
    assert rng.store(np.array([-3.0, 0.0, 5.0, 400.0, -400.0], np.float32), "e8m0").view(np.uint8).tolist() == [124, 127, 132, 254, 0]


def _mx_case(M, N, K, seed, lo=-3, hi=3):
    ch = replace(wl.gemm_mxf8_bias_gelu_scale_clamp(M, N, K, out_dtype="f32", exp_lo=lo, exp_hi=hi), ops=())
    return ch, wl.make_inputs(ch, seed)[:4]


def test_mx_gemm_unit_scales_is_the_plain_contraction(orc):
    ch, ins = _mx_case(6, 5, 96, 3)
    ones = [np.full(a.shape, 127, np.uint8).view(np.int8) for a in ins[2:4]]
    got = orc.run_chain(ch, ins[:2] + ones)["main"]
    assert np.array_equal(got, orc.gemm_nt(orc.widen(ins[0]), orc.widen(ins[1])))


def test_mx_gemm_single_block_is_a_diagonally_scaled_product(orc):
    """One block (K = 32): every row of A and of B has one scale, so V = diag(sa) (A B^T) diag(sb) exactly."""
    ch, ins = _mx_case(7, 9, 32, 4, lo=-20, hi=20)
    got = orc.run_chain(ch, ins)["main"]
    a, b, sa, sb = (orc.widen(t) for t in ins)
    assert np.array_equal(got, sa * (a @ b.T) * sb.T)       # powers of two: the scaling is exact in any order


def test_mx_gemm_block_boundaries(orc):
    """Operands that are one-hot at k = 31, 32 and 95: each product must pick up the scales of its own block
    (0, 1 and 2), which pins the block length and the index of the scale arrays."""
    M = N = 3
    K = 96
    a = np.zeros((M, K), np.float32)
    b = np.zeros((N, K), np.float32)
    ks = [31, 32, 95]
    for i, k in enumerate(ks):
        a[i, k] = 1.5
        b[:, k] = 2.0
    sa = np.array([[1, 2, 3], [4, 5, 6], [-1, -2, -3]], np.float32)
    sb = np.array([[0, 1, 0], [2, 0, -2], [7, 8, 9]], np.float32)
    got = orc.gemm_nt_mx(orc.widen(rng.store(a, "f8e4m3")), orc.widen(rng.store(b, "f8e4m3")),
                         orc.widen(rng.store(sa, "e8m0")), orc.widen(rng.store(sb, "e8m0")))
    want = np.array([[3.0 * 2.0 ** (sa[m, k // 32] + sb[n, k // 32]) for n in range(N)] for m, k in enumerate(ks)])
    assert np.array_equal(got, want)


def test_mx_gemm_brute_force_rationals(orc):
    from fractions import Fraction
    ch, ins = _mx_case(3, 4, 64, 5, lo=-6, hi=6)
    got = orc.run_chain(ch, ins)["main"]
    a, b, sa, sb = ([[Fraction(float(v)) for v in row] for row in orc.widen(t)] for t in ins)
    for n in reversed(range(4)):                 # a different loop order: columns outermost, blocks and k descending
        for m in range(3):
            acc = Fraction(0)
            for j in reversed(range(2)):
                for k in reversed(range(32 * j, 32 * j + 32)):
                    acc += sa[m][j] * sb[n][j] * a[m][k] * b[n][k]
            assert Fraction(float(got[m, n])) == acc
