"""Pins of the oracle's GPTQ error-compensation loop (Algorithm 1) against things other than itself:
the defining property of the factor, a column-by-column elimination written with scalar loops, the
constrained least-squares problem the update solves, and special cases with known answers."""
import numpy as np
import pytest

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl


def _layer(N, K, T, name="gptq", block=0):
    seed = wl.layer_seed("test", f"{name}-{N}x{K}", block)
    return wl.make_weight(seed, N, K), wl.make_calibration_x(seed, T, K)


def _w_hat(codes, scales, zeros, g=128):
    return orc.dequant_f64(codes, scales, zeros, g)


# ------------------------------------------------------------------------------------------ Hessian and factor
def test_hessian_is_the_token_average_of_outer_products():
    _, x = _layer(4, 256, 5)
    H = orc.gptq_hessian(x)
    want = np.zeros((256, 256))
    for t in range(5):
        v = x[t].astype(np.float64)
        want += np.outer(v, v)
    assert np.abs(H - want / 5).max() <= 1e-12 * np.abs(want).max()


def test_factor_defining_property_and_damping():
    _, x = _layer(4, 256, 64)                       # fewer tokens than channels: H alone is singular
    H = orc.gptq_hessian(x)
    U, dead = orc.gptq_factor(H, 0.01)
    assert not dead.any()
    assert np.abs(np.tril(U, -1)).max() == 0 and (np.diag(U) > 0).all()
    Hd = H + 0.01 * np.trace(H) / 256 * np.eye(256)
    assert np.abs(U.T @ U @ Hd - np.eye(256)).max() <= 1e-8
    # the factor of c H is U / sqrt(c): the 1/P of the Hessian cannot matter downstream
    U4, _ = orc.gptq_factor(4 * H, 0.01)
    assert np.abs(U4 * 2 - U).max() <= 1e-9 * np.abs(U).max()


# ------------------------------------------------------------------------------------------ the update
def _columnwise(W16, x16, codes, scales, zeros, lam, upto, g=128):
    """The published column-by-column elimination with the codes held fixed, scalar loops: after column k is set
    to its quantised value, its error divided by U_kk is pushed onto every later column through row k of U."""
    U, _ = orc.gptq_factor(orc.gptq_hessian(x16), lam)
    w = W16.astype(np.float64).copy()
    w_hat = _w_hat(codes, scales, zeros, g)
    N, K = w.shape
    for k in range(upto):
        for n in range(N):
            e = (w[n, k] - w_hat[n, k]) / U[k, k]
            for k2 in range(k + 1, K):
                w[n, k2] -= e * U[k, k2]
    return w


def test_block_update_equals_column_by_column_elimination():
    W, x = _layer(3, 384, 40, name="gptq-col")
    bits = np.array([2, 3, 1])
    for quantizer in ("minmax", "sqc"):
        codes, scales, zeros, w_run = orc.gptq_quantize(W, x, bits, 0.01, quantizer)
        # what both forms define is the weights a group is quantised FROM: for the last group, the running
        # columns after the elimination has passed the 256 columns of the first two groups
        w_in = _columnwise(W, x, codes, scales, zeros, 0.01, 256)[:, 256:]
        assert np.abs(w_run[:, 256:] - w_in).max() <= 1e-9
        w_mid = _columnwise(W, x, codes, scales, zeros, 0.01, 128)[:, 128:256]       # the same for the second group
        q1 = (orc.quantize_minmax if quantizer == "minmax" else (lambda a, b: orc.quantize_sqc(a, b)[:3]))(w_mid.astype(np.float16), bits[1:2])
        assert (q1[0] == codes[:, 128:256]).all()
        # and the codes of the last group are the quantizer's on exactly those weights
        q_fn = orc.quantize_minmax if quantizer == "minmax" else (lambda a, b: orc.quantize_sqc(a, b)[:3])
        q, s, z = q_fn(w_in.astype(np.float16), bits[2:3])
        assert (q == codes[:, 256:]).all() and (s[0] == scales[2]).all() and (z[0] == zeros[2]).all()


@pytest.mark.parametrize("g", [32, 64, 256])
def test_block_update_equals_column_by_column_elimination_at_other_group_sizes(g):
    """Algorithm 1 takes blocks of beta columns: with groups of g columns the block update over a group must still
    equal the column-by-column elimination over its g columns."""
    K = 3 * g
    W, x = _layer(2, K, 40 if g < 256 else 900, name=f"gptq-col-g{g}")
    bits = np.array([2, 3, 1])
    for quantizer in ("minmax", "sqc"):
        codes, scales, zeros, w_run = orc.gptq_quantize(W, x, bits, 0.01, quantizer, g)
        w_in = _columnwise(W, x, codes, scales, zeros, 0.01, 2 * g, g)[:, 2 * g:]
        assert np.abs(w_run[:, 2 * g:] - w_in).max() <= 1e-9
        q_fn = orc.quantize_minmax if quantizer == "minmax" else (lambda a, b, gg: orc.quantize_sqc(a, b, gg)[:3])
        q, s, z = q_fn(w_in.astype(np.float16), bits[2:3], g)
        assert (q == codes[:, 2 * g:]).all() and (s[0] == scales[2]).all() and (z[0] == zeros[2]).all()


def test_update_solves_the_constrained_least_squares_problem():
    """With the first groups fixed at their quantised values, the running weights of the other columns minimise
    ||(w' - w) x^T||^2 + lambda ||w' - w||^2 (the damped layer-output error) -- solved here with lstsq."""
    W, x = _layer(4, 384, 50, name="gptq-ls")
    bits = np.array([2, 2, 3])
    lam = 0.02
    H = orc.gptq_hessian(x)
    lam_abs = lam * np.trace(H) / 384
    codes, scales, zeros, _ = orc.gptq_quantize(W, x, bits, lam, "minmax")
    w_hat = _w_hat(codes, scales, zeros)
    w0 = W.astype(np.float64)
    X = x.astype(np.float64) / np.sqrt(x.shape[0])
    A = np.vstack([X, np.sqrt(lam_abs) * np.eye(384)])            # ||d A^T||^2 = d (H + lam I) d^T
    for fixed in (128, 256):
        # d = w' - w with d[:, :fixed] given; minimise over d[:, fixed:]
        d_fixed = w_hat[:, :fixed] - w0[:, :fixed]
        rhs = -(A[:, :fixed] @ d_fixed.T)
        d_free = np.linalg.lstsq(A[:, fixed:], rhs, rcond=None)[0].T
        # the oracle's running weights right after `fixed` columns: rerun the loop on the first groups only
        U, _ = orc.gptq_factor(H, lam)
        w = w0.copy()
        for j in range(fixed // 128):
            c = slice(128 * j, 128 * j + 128)
            E = (w[:, c] - w_hat[:, c]) @ np.linalg.inv(U[c, c])
            w[:, 128 * j + 128:] -= E @ U[c, 128 * j + 128:]
        assert np.abs((w[:, fixed:] - w0[:, fixed:]) - d_free).max() <= 1e-7 * max(1.0, np.abs(d_free).max())
    # ... and the loop inside gptq_quantize is that recursion: its last group was quantised from w[:, 256:]
    q, s, z = orc.quantize_minmax(w[:, 256:].astype(np.float16), bits[2:3])
    assert (q == codes[:, 256:]).all()


# ------------------------------------------------------------------------------------------ special cases
def test_uncorrelated_inputs_need_no_compensation():
    # x^T x = c I: the factor is diagonal, nothing is pushed onto other columns, the result is the plain quantizer's
    K = 256
    x = (np.eye(K) * 3.0).astype(np.float16)
    W = wl.make_weight(wl.layer_seed("test", "gptq-eye", 0), 8, K)
    bits = np.array([2, 3])
    for quantizer, plain in (("minmax", orc.quantize_minmax), ("sqc", lambda a, b: orc.quantize_sqc(a, b)[:3])):
        codes, scales, zeros, w_run = orc.gptq_quantize(W, x, bits, 0.01, quantizer)
        q, s, z = plain(W, bits)
        assert (codes == q).all() and (scales == s).all() and (zeros == z).all()
        assert np.abs(w_run - W.astype(np.float64)).max() == 0


def test_first_group_sees_the_original_weights_and_a_dead_channel_is_zeroed():
    W, x = _layer(6, 256, 32, name="gptq-dead")
    x = x.copy()
    x[:, 5] = 0
    bits = np.array([3, 2])
    codes, scales, zeros, _ = orc.gptq_quantize(W, x, bits, 0.01, "minmax")
    Wz = W.copy()
    Wz[:, 5] = 0
    q, s, z = orc.quantize_minmax(Wz[:, :128], bits[:1])
    assert (codes[:, :128] == q).all() and (scales[0] == s[0]).all()
    assert (_w_hat(codes, scales, zeros)[:, 5] == 0).all()


def test_compensation_lowers_the_layer_output_error():
    W, x = _layer(64, 512, 256, name="gptq-loss")
    for avg, bits in ((2, np.array([2, 1, 3, 2])), (3, np.array([3, 3, 3, 3]))):
        for quantizer, plain in (("minmax", orc.quantize_minmax), ("sqc", lambda a, b: orc.quantize_sqc(a, b)[:3])):
            codes, scales, zeros, _ = orc.gptq_quantize(W, x, bits, 0.01, quantizer)
            with_c = orc.gptq_proxy_loss(W, _w_hat(codes, scales, zeros), x)
            without = orc.gptq_proxy_loss(W, _w_hat(*plain(W, bits)), x)
            assert with_c < 0.8 * without, (avg, quantizer, with_c, without)


def test_scale_of_the_calibration_data_does_not_matter():
    W, x = _layer(8, 256, 40, name="gptq-scale")
    bits = np.array([2, 3])
    a = orc.gptq_quantize(W, x, bits, 0.01, "sqc")
    b = orc.gptq_quantize(W, (x.astype(np.float32) * 4).astype(np.float16), bits, 0.01, "sqc")      # exact in fp16
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all() and (a[2] == b[2]).all()
