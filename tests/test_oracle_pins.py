"""Pins for the CPU oracle: each operator is checked against something other than itself —
a second brute-force evaluation written differently (other loop order, float64), a library
matmul, closed forms on constant inputs, impulse responses, and the identities the paper
states (Eq. 1; "equivalent to the original model", Section 3)."""
import itertools

import numpy as np
import pytest

import oracle as xo
from xenos_workloads import gen


def brute_conv(x, w, b, stride, pad, groups):
    """Direct definition, loops ordered s, r, c outermost, float64 accumulation."""
    N, C, H, W = x.shape
    K, Cg, R, S = w.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = np.zeros((N, K, P, Q), np.float64)
    Kg = K // groups
    for s in range(S):
        for r in range(R):
            for c in range(Cg):
                for k in range(K):
                    ci = (k // Kg) * Cg + c
                    for n in range(N):
                        for p in range(P):
                            ih = p * stride - pad + r
                            if not 0 <= ih < H:
                                continue
                            for q in range(Q):
                                iw = q * stride - pad + s
                                if 0 <= iw < W:
                                    y[n, k, p, q] += float(x[n, ci, ih, iw]) * float(w[k, c, r, s])
    if b is not None:
        y += b.astype(np.float64)[None, :, None, None]
    return y


CASES = [
    # N, C, H, W, K, k, stride, pad, groups
    (2, 4, 7, 7, 6, 3, 1, 1, 1),
    (1, 4, 7, 6, 4, 3, 2, 1, 1),
    (1, 3, 7, 7, 2, 7, 2, 3, 1),
    (2, 4, 5, 5, 4, 3, 1, 1, 4),      # depthwise
    (1, 4, 6, 7, 4, 3, 2, 1, 4),      # depthwise, stride 2
    (1, 4, 5, 4, 3, 1, 1, 0, 1),
    (1, 4, 6, 6, 8, 1, 2, 0, 1),      # strided 1x1 (projection)
    (1, 4, 6, 6, 4, 3, 2, 0, 2),      # two groups, no pad
    (1, 2, 5, 5, 2, 5, 1, 2, 1),
]


@pytest.mark.parametrize("case", CASES)
def test_conv_matches_brute_force(case):
    N, C, H, W, K, k, st, pad, g = case
    x = gen.uniform(7, 0, (N, C, H, W), -1, 1)
    w = gen.normal(7, 1, (K, C // g, k, k), 0, 0.5)
    b = gen.uniform(7, 2, (K,), -0.1, 0.1)
    y = xo.conv2d(x, w, b, st, pad, g)
    ref = brute_conv(x, w, b, st, pad, g)
    assert y.shape == ref.shape
    np.testing.assert_allclose(y, ref, rtol=0, atol=2e-6 * max(1.0, np.abs(ref).max()))


def test_conv1x1_equals_matmul():
    N, C, H, W, K = 2, 24, 5, 7, 10
    x = gen.uniform(11, 0, (N, C, H, W), -1, 1)
    w = gen.normal(11, 1, (K, C, 1, 1), 0, 0.3)
    y = xo.conv2d(x, w)
    # library matmul in float64
    ref = np.einsum("kc,nchw->nkhw", w[:, :, 0, 0].astype(np.float64), x.astype(np.float64))
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-5)
    # textbook triple loop with the same ascending-c fp32 summation order: bit-exact
    x2 = x[0].reshape(C, H * W)
    acc = np.zeros((K, H * W), np.float32)
    for c in range(C):
        acc = acc + (w[:, c, 0, 0][:, None] * x2[c][None, :]).astype(np.float32)
    assert np.array_equal(y[0].reshape(K, H * W), acc)


def test_fc_equals_matmul_and_eq1_split():
    x = gen.uniform(3, 0, (5, 37), -1, 1)
    w = gen.normal(3, 1, (11, 37), 0, 0.2)
    b = gen.uniform(3, 2, (11,), -0.1, 0.1)
    y = xo.fc(x, w, b)
    np.testing.assert_allclose(y, x.astype(np.float64) @ w.T.astype(np.float64) + b, atol=1e-5, rtol=0)
    # Eq. 1: W -> (W1; W2), B -> (B1; B2); joined outputs equal the unsplit result exactly
    y1, y2 = xo.fc(x, w[:4], b[:4]), xo.fc(x, w[4:], b[4:])
    assert np.array_equal(np.concatenate([y1, y2], 1), y)


def test_conv_outc_split_is_exact():
    x = gen.uniform(5, 0, (2, 6, 9, 8), -1, 1)
    w = gen.normal(5, 1, (10, 6, 3, 3), 0, 0.2)
    b = gen.uniform(5, 2, (10,), -0.1, 0.1)
    y = xo.conv2d(x, w, b, 1, 1)
    parts = [xo.conv2d(x, w[a:c], b[a:c], 1, 1) for a, c in ((0, 3), (3, 4), (4, 10))]
    assert np.array_equal(np.concatenate(parts, 1), y)


def test_closed_forms_constant_inputs():
    a, bb = 0.75, -0.5
    C, K = 6, 4
    x = np.full((1, C, 6, 6), a, np.float32)
    w = np.full((K, C, 3, 3), bb, np.float32)
    bias = np.arange(K, dtype=np.float32)
    # no padding: a*b*C*R*S + bias
    y = xo.conv2d(x, w, bias, 1, 0)
    assert y.shape == (1, K, 4, 4)
    for k in range(K):
        np.testing.assert_allclose(y[0, k], a * bb * C * 9 + k, rtol=1e-6)
    # zero padding 1: corners see 4 taps, edges 6, interior 9
    y = xo.conv2d(x, w, None, 1, 1)
    taps = np.full((6, 6), 9.0)
    taps[0, :] = taps[-1, :] = taps[:, 0] = taps[:, -1] = 6.0
    taps[0, 0] = taps[0, -1] = taps[-1, 0] = taps[-1, -1] = 4.0
    np.testing.assert_allclose(y[0, 0], a * bb * C * taps, rtol=1e-6)
    # depthwise: a*b*9 in the interior
    wd = np.full((C, 1, 3, 3), bb, np.float32)
    y = xo.conv2d(x, wd, None, 1, 1, groups=C)
    np.testing.assert_allclose(y[0, :, 1:-1, 1:-1], a * bb * 9, rtol=1e-6)
    # pools and pointwise ops on constants
    assert np.all(xo.maxpool(x, 3, 2, 1) == a)
    assert np.all(xo.maxpool(x, 2, 2, 0) == a)
    np.testing.assert_allclose(xo.avgpool(x, 2, 2, 0), a, rtol=1e-6)
    np.testing.assert_allclose(xo.global_avgpool(x), a, rtol=1e-6)
    assert np.all(xo.add(x, x) == 2 * a)
    assert np.all(xo.relu6(np.full((4,), 7.0, np.float32)) == 6.0)
    assert np.all(xo.relu(np.full((4,), -7.0, np.float32)) == 0.0)
    assert np.all(xo.relu6(np.full((4,), 2.5, np.float32)) == 2.5)
    # BN at x == mean returns beta
    mean = np.linspace(-1, 1, C).astype(np.float32)
    xm = np.broadcast_to(mean[None, :, None, None], (1, C, 3, 3)).copy()
    beta = np.linspace(0.1, 0.6, C).astype(np.float32)
    y = xo.batchnorm(xm, np.full(C, 1.3, np.float32), beta, mean, np.full(C, 0.7, np.float32))
    assert np.array_equal(y, np.broadcast_to(beta[None, :, None, None], y.shape))


def test_impulse_returns_flipped_kernel():
    C, K, k = 3, 2, 3
    w = gen.normal(9, 1, (K, C, k, k), 0, 1)
    for c in range(C):
        x = np.zeros((1, C, 5, 5), np.float32)
        x[0, c, 2, 2] = 1.0
        y = xo.conv2d(x, w, None, 1, 1)
        # y[k][p][q] = w[k][c][2-p+1][2-q+1] on the 3x3 neighbourhood of the impulse
        for kk in range(K):
            assert np.array_equal(y[0, kk, 1:4, 1:4], w[kk, c, ::-1, ::-1])
    # a transposed kernel or swapped r/s would fail the asymmetric check above; and stride 2:
    x = np.zeros((1, 1, 7, 7), np.float32)
    x[0, 0, 3, 4] = 1.0
    w1 = gen.normal(9, 2, (1, 1, 3, 3), 0, 1)
    y = xo.conv2d(x, w1, None, 2, 1)          # out 4x4; taps: ih = 2p-1+r == 3, iw = 2q-1+s == 4
    exp = np.zeros((4, 4), np.float32)
    for p in range(4):
        for q in range(4):
            r, s = 3 - (2 * p - 1), 4 - (2 * q - 1)
            if 0 <= r < 3 and 0 <= s < 3:
                exp[p, q] = w1[0, 0, r, s]
    assert np.array_equal(y[0, 0], exp)


def test_bn_fold_equals_conv_then_bn():
    x = gen.uniform(13, 0, (2, 5, 6, 6), -1, 1)
    w = gen.normal(13, 1, (7, 5, 3, 3), 0, 0.3)
    g_ = gen.uniform(13, 2, (7,), 0.5, 1.5)
    be = gen.uniform(13, 3, (7,), -0.1, 0.1)
    mu = gen.normal(13, 4, (7,), 0, 0.1)
    var = gen.uniform(13, 5, (7,), 0.5, 1.5)
    y = xo.batchnorm(xo.conv2d(x, w, None, 1, 1), g_, be, mu, var, 1e-5)
    scale = g_.astype(np.float64) / np.sqrt(var.astype(np.float64) + 1e-5)
    wf = (w.astype(np.float64) * scale[:, None, None, None]).astype(np.float32)
    bf = (be.astype(np.float64) - mu.astype(np.float64) * scale).astype(np.float32)
    yf = xo.conv2d(x, wf, bf, 1, 1)
    np.testing.assert_allclose(yf, y, rtol=0, atol=4e-6 * np.abs(y).max())


def test_bn_matches_float64_definition():
    x = gen.uniform(17, 0, (2, 4, 3, 3), -2, 2)
    g_, be = gen.uniform(17, 1, (4,), 0.5, 1.5), gen.uniform(17, 2, (4,), -0.1, 0.1)
    mu, var = gen.normal(17, 3, (4,), 0, 0.1), gen.uniform(17, 4, (4,), 0.5, 1.5)
    y = xo.batchnorm(x, g_, be, mu, var, 1e-5)
    sh = (1, 4, 1, 1)
    ref = g_.reshape(sh).astype(np.float64) * (x - mu.reshape(sh)) / np.sqrt(var.reshape(sh) + 1e-5) + be.reshape(sh)
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-6)


def test_pools_against_numpy_windows():
    x = gen.uniform(19, 0, (2, 3, 9, 8), -1, 0)   # all negative: zero padding must never win a max
    for k, st, pad in ((3, 2, 1), (3, 2, 0), (2, 2, 0)):
        y = xo.maxpool(x, k, st, pad)
        ya = xo.avgpool(x, k, st, pad)
        P, Q = y.shape[2:]
        for p, q in itertools.product(range(P), range(Q)):
            h0, h1 = max(0, p * st - pad), min(9, p * st - pad + k)
            w0, w1 = max(0, q * st - pad), min(8, q * st - pad + k)
            win = x[:, :, h0:h1, w0:w1]
            assert np.array_equal(y[:, :, p, q], win.max(axis=(2, 3)))
            np.testing.assert_allclose(ya[:, :, p, q], win.astype(np.float64).mean(axis=(2, 3)), atol=1e-6)
    assert np.all(xo.maxpool(x, 3, 2, 1) < 0)
    np.testing.assert_allclose(xo.global_avgpool(x), x.astype(np.float64).mean(axis=(2, 3)), atol=1e-6)


def test_concat_and_add_and_round():
    a = gen.index_valued((2, 3, 2, 2))
    b = gen.index_valued((2, 5, 2, 2), 97) + 1000
    y = xo.concat([a, b])
    assert np.array_equal(y, np.concatenate([a, b], 1))
    assert np.array_equal(xo.add(a, a * 2), a * 3)
    # bf16 rounding: ties to even on the 16th mantissa bit
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -3.1415926], np.float32)
    r = xo.round_bf16(v)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == 1.0 + 2 ** -6
    assert abs(r[4] + 3.140625) < 1e-7


def _stages():
    w3 = gen.normal(23, 1, (8, 4, 3, 3), 0, 0.3)
    w1 = gen.normal(23, 2, (6, 8, 1, 1), 0, 0.3)
    bn1 = (gen.uniform(23, 3, (8,), .5, 1.5), gen.uniform(23, 4, (8,), -.1, .1),
           gen.normal(23, 5, (8,), 0, .1), gen.uniform(23, 6, (8,), .5, 1.5), 1e-5)
    bn2 = (gen.uniform(23, 7, (6,), .5, 1.5), gen.uniform(23, 8, (6,), -.1, .1),
           gen.normal(23, 9, (6,), 0, .1), gen.uniform(23, 10, (6,), .5, 1.5), 1e-5)
    return w3, w1, bn1, bn2


@pytest.mark.parametrize("tile", [(1, 1), (2, 3), (4, 4), (5, 7), (64, 64)])
def test_linked_tiles_equal_unlinked_bit_exact(tile):
    """Section 3: the optimised model is equivalent to the original one."""
    w3, w1, bn1, bn2 = _stages()
    x = gen.uniform(23, 0, (2, 4, 13, 11), -1, 1)
    y = xo.relu(xo.batchnorm(xo.conv2d(x, w3, None, 1, 1), *bn1))
    y = xo.relu(xo.batchnorm(xo.conv2d(y, w1), *bn2))
    y = xo.maxpool(y, 2, 2, 0)
    st = [dict(kind="conv", w=w3, stride=1, pad=1, bn=bn1, act="relu"),
          dict(kind="conv", w=w1, bn=bn2, act="relu"),
          dict(kind="maxpool", k=2, stride=2, pad=0)]
    yt = xo.chain_tiled(x, st, *tile)
    assert np.array_equal(yt, y)


def test_linked_conv3_conv3_stride2_and_dw_chain():
    x = gen.uniform(29, 0, (1, 4, 12, 10), -1, 1)
    wa = gen.normal(29, 1, (4, 1, 3, 3), 0, 0.4)          # depthwise, stride 2
    wb = gen.normal(29, 2, (5, 4, 3, 3), 0, 0.3)
    bb = gen.uniform(29, 3, (5,), -.1, .1)
    y = xo.relu6(xo.conv2d(x, wa, None, 2, 1, groups=4))
    y = xo.conv2d(y, wb, bb, 1, 1)
    y = xo.maxpool(y, 3, 2, 1)
    st = [dict(kind="conv", w=wa, stride=2, pad=1, groups=4, act="relu6"),
          dict(kind="conv", w=wb, bias=bb, stride=1, pad=1),
          dict(kind="maxpool", k=3, stride=2, pad=1)]
    for tile in ((1, 2), (2, 2), (3, 1)):
        assert np.array_equal(xo.chain_tiled(x, st, *tile), y)


def test_halo_equals_brute_force_receptive_field():
    """Section 4.2.1: inH/inW partitions need the boundary rows/columns of their neighbours."""
    w3, w1, bn1, bn2 = _stages()
    x = gen.uniform(31, 0, (1, 4, 16, 16), -1, 1)
    st = [dict(kind="conv", w=w3, stride=1, pad=1), dict(kind="conv", w=w1),
          dict(kind="maxpool", k=2, stride=2, pad=0)]
    th, tw = 3, 2
    y0, halo = xo.chain_tiled(x, st, th, tw, want_halo=True)
    # brute force: perturb each input position, see whether tile (0,0) of the output changes
    touched = np.zeros((16, 16), bool)
    for i in range(16):
        for j in range(16):
            xp = x.copy()
            xp[0, :, i, j] += 1.0
            y = xo.maxpool(xo.conv2d(xo.conv2d(xp, w3, None, 1, 1), w1), 2, 2, 0)
            yb = xo.maxpool(xo.conv2d(xo.conv2d(x, w3, None, 1, 1), w1), 2, 2, 0)
            touched[i, j] = not np.array_equal(y[0, :, :th, :tw], yb[0, :, :th, :tw])
    rows = np.where(touched.any(1))[0]
    cols = np.where(touched.any(0))[0]
    assert (rows.min(), rows.max() + 1, cols.min(), cols.max() + 1) == tuple(halo[0])
    assert tuple(halo[2]) == (0, 2 * th, 0, 2 * tw)


def test_generator_is_deterministic_and_in_range():
    a = gen.uniform(1, 5, (1000,), -1, 1)
    assert np.array_equal(a, gen.uniform(1, 5, (1000,), -1, 1))
    assert not np.array_equal(a, gen.uniform(1, 6, (1000,), -1, 1))
    assert not np.array_equal(a, gen.uniform(2, 5, (1000,), -1, 1))
    assert a.min() > -1 and a.max() < 1 and abs(a.mean()) < 0.1
    z = gen.normal(1, 5, (20000,), 0.0, 2.0)
    assert abs(z.mean()) < 0.06 and abs(z.std() - 2.0) < 0.06


# ---- the remaining operators of Table 3: x.mul, x.mac, x.transpose, x.split, x.matmul ------------------
def test_mul_and_mac_against_numpy_and_the_rounded_product():
    a = gen.uniform(7, 1, (2, 3, 4, 5), -2.0, 2.0)
    b = gen.uniform(7, 2, (2, 3, 4, 5), -2.0, 2.0)
    c = gen.uniform(7, 3, (2, 3, 4, 5), -2.0, 2.0)
    assert np.array_equal(xo.mul(a, b), a * b)
    assert np.array_equal(xo.mac(a, b, c), (a * b).astype(np.float32) + c)
    # the product is rounded before the sum: (1 + 2^-12)^2 = 1 + 2^-11 + 2^-24 rounds to 1 + 2^-11 (a tie, to even),
    # so adding -(1 + 2^-11) gives exactly 0; a fused multiply-add would leave 2^-24
    one = np.full((1, 1, 1, 1), 1.0 + 2.0 ** -12, np.float32)
    neg = np.full((1, 1, 1, 1), -(1.0 + 2.0 ** -11), np.float32)
    assert xo.mac(one, one, neg)[0, 0, 0, 0] == 0.0
    # swapped roles change the result: a * c + b differs from a * b + c
    assert not np.array_equal(xo.mac(a, b, c), xo.mac(a, c, b))


def test_transpose_is_the_index_swap_and_an_involution():
    N, C, H = 2, 5, 7
    x = np.arange(N * C * H, dtype=np.float32).reshape(N, C, H, 1)
    y = xo.transpose(x)
    assert y.shape == (N, H, C, 1)
    for n, c, h in itertools.product(range(N), range(C), range(H)):
        assert y[n, h, c, 0] == x[n, c, h, 0]
    assert np.array_equal(xo.transpose(y), x)


def test_split_parts_are_slices_and_concat_restores_the_tensor():
    x = np.arange(2 * 10 * 3 * 4, dtype=np.float32).reshape(2, 10, 3, 4)
    parts = [(0, 3), (3, 5), (8, 2)]
    ys = [xo.split_part(x, f, n) for f, n in parts]
    for (f, n), y in zip(parts, ys):
        assert np.array_equal(y, x[:, f:f + n])
    assert np.array_equal(xo.concat(ys), x)


def test_matmul_against_float64_identity_and_fc():
    N, K, R, M = 2, 9, 6, 5
    a = gen.uniform(11, 1, (N, K, R, 1), -1.0, 1.0)
    b = gen.normal(11, 2, (K, M), 0.0, 0.5)
    bias = gen.uniform(11, 3, (M,), -0.1, 0.1)
    y = xo.matmul(a, b, bias)
    ref = np.einsum("nkr,km->nmr", a[..., 0].astype(np.float64), b.astype(np.float64)) + bias.astype(np.float64)[None, :, None]
    assert y.shape == (N, M, R, 1) and np.abs(y[..., 0] - ref).max() <= 1e-5
    # B = identity returns A
    assert np.array_equal(xo.matmul(a, np.eye(K, dtype=np.float32)), a)
    # a vector times B is Eq. 1 with W = B^T: same products, same order of the sum
    v = gen.uniform(11, 4, (N, K), -1.0, 1.0)
    assert np.array_equal(xo.matmul(v, b, bias), xo.fc(v, np.ascontiguousarray(b.T), bias))
    # (A B1) B2 = A (B1 B2) within rounding: the identity the MatmulX -> MatmulY link rests on
    b2 = gen.normal(11, 5, (M, 4), 0.0, 0.5)
    two = xo.matmul(xo.matmul(a, b), b2)
    one = xo.matmul(a, (b.astype(np.float64) @ b2.astype(np.float64)).astype(np.float32))
    assert np.abs(two - one).max() <= 1e-5 * max(1.0, np.abs(two).max())
