"""Shared helpers of the GPU parity tests: seeded layers through the oracle, tolerance checks."""
import numpy as np

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl

# acceptance bounds for y against the fp64 oracle (the benchmark spec)
MAX_ABS_REL = 5e-3   # max|y - y_ref| <= 5e-3 * max|y_ref|
FRO_REL = 1e-3       # ||y - y_ref||_F <= 1e-3 * ||y_ref||_F


def oracle_layer(N, K, avg_bits, M, seed_name="parity", block=0, bits=None, outliers=True):
    """Seeded layer quantised by the oracle.  Returns a dict of numpy arrays."""
    seed = wl.layer_seed("test", f"{seed_name}-{N}x{K}", block)
    W = wl.make_weight(seed, N, K, outlier_frac=0.01 if outliers else 0.0)
    a = wl.make_act_norms(seed, K)
    x = wl.make_x(seed, M, K)
    if bits is None:
        bits = orc.allocate_bits(orc.group_salience(W, a), avg_bits)
    bits = np.asarray(bits, dtype=np.uint8)
    codes, scales, zeros = orc.quantize_minmax(W, bits)
    return dict(W=W, a=a, x=x, bits=bits, codes=codes, scales=scales, zeros=zeros, N=N, K=K, M=M)


def check_output(y, y_ref, what=""):
    y = np.asarray(y, dtype=np.float64)
    assert np.isfinite(y).all(), f"{what}: non-finite output"
    max_ref = np.abs(y_ref).max()
    max_err = np.abs(y - y_ref).max()
    fro = np.linalg.norm(y - y_ref) / max(np.linalg.norm(y_ref), 1e-300)
    assert max_err <= MAX_ABS_REL * max_ref, f"{what}: max abs err {max_err:.3e} > {MAX_ABS_REL} * {max_ref:.3e}"
    assert fro <= FRO_REL, f"{what}: relative Frobenius error {fro:.3e} > {FRO_REL}"
    return max_err / max(max_ref, 1e-300), fro
