"""Pins of the SQC oracle (Sec. 3.3, Eq. 5, function SQC of Algorithm 2): a brute-force restatement
with plain Python floats, and properties the definition fixes."""
import struct

import numpy as np

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl


def _f16(v: float) -> float:
    try:
        return struct.unpack("<e", struct.pack("<e", v))[0]
    except OverflowError:
        return 65504.0


def _brute_sqc_row(w, b, lam=0.1, n=50):
    """One (row, group) exactly as Algorithm 2 lists it, scalar Python, no NumPy arithmetic."""
    levels = 2 ** b - 1
    wmin, wmax = min(min(w), 0.0), max(max(w), 0.0)
    mu = sum(w) / len(w)
    sd = (sum((v - mu) ** 2 for v in w) / len(w)) ** 0.5
    best = None
    for i in range(2 * n):
        tau = 1.0 - lam + i * (lam / n)
        delta = _f16(tau * (wmax - wmin) / levels)
        if delta == 0.0:
            delta = 1.0
        z = min(max(-round(tau * wmin / delta), 0), levels)
        q = [min(max(round(v / delta) + z, 0), levels) for v in w]
        Ls = Lus = 0.0
        for v, c in zip(w, q):
            e = v - delta * (c - z)
            if v < mu - 3.0 * sd or v > mu + 3.0 * sd:
                Ls += e * e
            else:
                Lus += e * e
        if best is None or Ls + Lus < best[0]:
            best = (Ls + Lus, i, delta, z, q, Ls)
    return best


def test_brute_force_agrees_on_small_layers():
    rng = np.random.default_rng(21)
    for b in (1, 2, 3, 4):
        W = (rng.standard_normal((3, 256)) * 0.02).astype(np.float16)
        W[0, 5] = np.float16(0.3)            # an outlier the 3-sigma mask must catch
        W[2, :128] = np.abs(W[2, :128])      # all-positive group
        bits = np.array([b, b], np.uint8)
        codes, scales, zeros, ti, loss, loss_s = orc.quantize_sqc(W, bits)
        for r in range(3):
            for j in range(2):
                w = [float(v) for v in W[r, 128 * j:128 * (j + 1)]]
                L, i, delta, z, q, Ls = _brute_sqc_row(w, b)
                assert ti[j, r] == i
                assert float(scales[j, r]) == delta and float(zeros[j, r]) == z
                assert list(codes[r, 128 * j:128 * (j + 1)]) == q
                assert loss[j, r] == L and loss_s[j, r] == Ls


def test_grid_contains_the_plain_quantizer_and_spans_the_interval():
    t = orc.sqc_tau_grid()
    assert t.shape == (100,) and abs(t[0] - 0.9) < 1e-15 and abs(t[50] - 1.0) < 1e-15 and abs(t[99] - 1.098) < 1e-12
    assert np.allclose(np.diff(t), 0.002, atol=1e-15)


def test_never_worse_than_min_max_and_loss_is_the_dequantisation_error():
    seed = wl.layer_seed("test", "sqc", 0)
    W = wl.make_weight(seed, 48, 1024)
    bits = np.array([1, 2, 3, 4, 2, 3, 1, 4], np.uint8)
    codes, scales, zeros, ti, loss, loss_s = orc.quantize_sqc(W, bits)
    err = (W.astype(np.float64) - orc.dequant_f64(codes, scales, zeros)) ** 2
    total = err.reshape(48, 8, 128).sum(axis=2).T
    assert np.allclose(total, loss, rtol=1e-12, atol=0)
    c0, s0, z0 = orc.quantize_minmax(W, bits)
    e0 = ((W.astype(np.float64) - orc.dequant_f64(c0, s0, z0)) ** 2).reshape(48, 8, 128).sum(axis=2).T
    assert (loss <= e0 * (1 + 1e-12)).all()          # tau = 1 is a candidate
    assert (loss_s <= loss).all() and (loss_s >= 0).all()
    # codes stay inside their group's range, zero points are integers in range
    for j, b in enumerate(bits):
        assert codes[:, 128 * j:128 * (j + 1)].max() < 2 ** int(b)
        zz = zeros[j].astype(np.float64)
        assert (zz == np.rint(zz)).all() and zz.min() >= 0 and zz.max() <= 2 ** int(b) - 1


def test_weights_on_the_grid_of_tau_one_are_reproduced_exactly():
    rng = np.random.default_rng(4)
    for b in (2, 3, 4):
        levels = 2 ** b - 1
        z = levels // 2
        q = rng.integers(0, levels + 1, (4, 128))
        q[:, 0], q[:, 1] = 0, levels                   # the range is attained: Delta(tau = 1) = 0.25
        W = (0.25 * (q - z)).astype(np.float16)
        codes, scales, zeros, ti, loss, _ = orc.quantize_sqc(W, np.array([b], np.uint8))
        assert (loss == 0).all() and (ti == 50).all()
        assert (codes == q).all() and (scales == np.float16(0.25)).all() and (zeros == z).all()


def test_mask_selects_planted_outliers_and_scaling_by_two_changes_only_the_scale():
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((8, 256)) * 0.01).astype(np.float16)
    W[:, 17] = np.float16(0.5)
    m = orc.salient_mask_3sigma(W)
    assert m[:, 17].all() and m.mean() < 0.05
    bits = np.array([2, 3], np.uint8)
    a = orc.quantize_sqc(W, bits)
    b2 = orc.quantize_sqc((W.astype(np.float32) * 2).astype(np.float16), bits)
    assert (a[0] == b2[0]).all() and (a[3] == b2[3]).all() and (a[2] == b2[2]).all()
    assert (b2[1].astype(np.float32) == 2 * a[1].astype(np.float32)).all()
