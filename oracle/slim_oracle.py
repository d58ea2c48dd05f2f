"""CPU oracle for the group-wise mixed-precision weight-only linear layer.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
statement of what the CUDA library must compute.  It shares no code with the
CUDA path and must never be imported by it: only the tests, the smoke check and
the CPU-baseline leg of the benchmark may call it.

Notation follows the paper: the weight is w in R^{n x m} (here N x K, groups of
g = 128 consecutive input columns, Algorithm 1 slices w[:, b:b+beta]), x in
R^{t x m} (here M x K), N-bar is the target average bit-width.

Everything floating point is fp64 computed from fp16-exact inputs unless a line
says otherwise.

Pinned (tests/test_oracle_*.py): bit budget, quantizer closed forms and brute
force, packing positions, dequantisation single-rounding, linear layer special
cases, the SQC line search (brute force, never worse than tau = 1, exact grids), the SBA search
(library KL, shift invariance, constructed optima, budget), the GPTQ loop (column-by-column
elimination, constrained least squares, H = I, proxy loss).  Parity unpinned: nothing in this file (the paper's perplexity / accuracy
/ token-per-second tables are not reproduced at all).
"""
from __future__ import annotations

import numpy as np

GROUP = 128

# A b-bit code is stored as slices (lo, w): slice value = (q >> lo) & (2^w - 1).
# This is the storage format's definition, restated here independently.
CODE_SLICES = {1: ((0, 1),), 2: ((0, 2),), 3: ((0, 2), (2, 1)), 4: ((0, 4),)}


# --------------------------------------------------------------------------- salience / bit map
def group_salience(W16: np.ndarray, act_norm: np.ndarray, g: int = GROUP, power: int = 2) -> np.ndarray:
    """Group salience S_j = sum_{k in group j} a_k^power * sum_n w[n,k]^2.

    Diagonal form of Definition 1 / Theorem 1 (Sec. 3.2.1): the salience of a
    column is proportional to its squared weights times the squared activation
    norm of that input channel.  Alg. 2 (SBA, first step) averages it per group;
    sum and average rank groups identically because groups have equal size.
    """
    W = W16.astype(np.float64)
    a = np.asarray(act_norm).astype(np.float64)
    N, K = W.shape
    assert K % g == 0 and a.shape == (K,)
    col = (W * W).sum(axis=0) * a**power
    return col.reshape(K // g, g).sum(axis=1)


def allocate_bits(salience: np.ndarray, avg_bits: int, p: int | None = None) -> np.ndarray:
    """Bit-width per group under the constraint |G_{N-1}| = |G_{N+1}| (Eq. 4).

    Groups are ranked by salience (descending; equal salience: lower index first).
    The p most salient groups get N-bar+1 bits, the p least salient N-bar-1, the
    rest N-bar.  p defaults to floor(G/4), the fixed ratio of the benchmark
    workloads (the paper searches p with a KL objective, Alg. 2).
    """
    S = np.asarray(salience, dtype=np.float64)
    G = S.shape[0]
    if p is None:
        p = G // 4
    assert 0 <= 2 * p <= G
    order = sorted(range(G), key=lambda j: (-S[j], j))
    bits = np.full(G, avg_bits, dtype=np.uint8)
    for j in order[:p]:
        bits[j] = avg_bits + 1
    for j in order[G - p:] if p > 0 else []:
        bits[j] = avg_bits - 1
    return bits


# --------------------------------------------------------------------------- quantizer (Eq. 1)
def quantize_minmax(W16: np.ndarray, bits: np.ndarray, g: int = GROUP):
    """Asymmetric min-max uniform quantizer of Eq. 1, per (row, group).

        s = (w_max - w_min) / (2^b - 1),  z = -round(w_min / s),
        q = clamp(round(w / s) + z, 0, 2^b - 1)

    Readings where the paper is silent: round = round-half-to-even; the range
    always contains 0 (w_min <= 0 <= w_max) so that z lies in [0, 2^b - 1]; the
    scale is rounded to fp16 (stored format) *before* z and q are computed; a
    zero scale becomes 1; a scale beyond the fp16 range becomes 65504.

    Returns codes uint8 [N][K], scales fp16 [G][N], zeros fp16 [G][N].
    """
    N, K = W16.shape
    G = K // g
    assert K % g == 0 and len(bits) == G
    codes = np.zeros((N, K), dtype=np.uint8)
    scales = np.zeros((G, N), dtype=np.float16)
    zeros = np.zeros((G, N), dtype=np.float16)
    for j in range(G):
        b = int(bits[j])
        levels = float(2**b - 1)
        w = W16[:, j * g:(j + 1) * g].astype(np.float64)
        lo = np.minimum(w.min(axis=1), 0.0)
        hi = np.maximum(w.max(axis=1), 0.0)
        with np.errstate(over="ignore"):
            s16 = ((hi - lo) / levels).astype(np.float16)
        s16[np.isinf(s16)] = np.float16(65504.0)
        s16[s16 == 0] = np.float16(1.0)
        s = s16.astype(np.float64)
        z = np.clip(-np.rint(lo / s), 0.0, levels) + 0.0   # an unsigned integer: -0.0 is stored as +0
        q = np.clip(np.rint(w / s[:, None]) + z[:, None], 0.0, levels)
        codes[:, j * g:(j + 1) * g] = q.astype(np.uint8)
        scales[j] = s16
        zeros[j] = z.astype(np.float16)
    return codes, scales, zeros


def sqc_tau_grid(lam: float = 0.1, n: int = 50) -> np.ndarray:
    """Calibration candidates of SQC (Sec. 3.3): [1 - lam, 1 + lam] cut into 2n slices.

    Reading: the 2n candidates are the left ends of the slices, tau_i = 1 - lam + i * lam / n for
    i = 0 .. 2n-1, so tau = 1 (the plain min-max quantizer) is candidate n.
    """
    return 1.0 - lam + np.arange(2 * n, dtype=np.float64) * (lam / n)


def salient_mask_3sigma(W16: np.ndarray, g: int = GROUP) -> np.ndarray:
    """3-sigma mask of Sec. 3.3 per (row, group): w < mu - 3 sigma or w > mu + 3 sigma, with mu and
    sigma the mean and (population) standard deviation of the group's 128 weights.  Both sums run
    in column order (the paper fixes no order; a fixed one lets every implementation agree on
    which elements sit exactly at the threshold)."""
    N, K = W16.shape
    w = W16.astype(np.float64).reshape(N, K // g, g)
    tot = np.zeros((N, K // g))
    for k in range(g):
        tot = tot + w[:, :, k]
    mu = tot / g
    var = np.zeros((N, K // g))
    for k in range(g):
        d = w[:, :, k] - mu
        var = var + d * d
    sd = np.sqrt(var / g)
    lo, hi = (mu - 3.0 * sd)[:, :, None], (mu + 3.0 * sd)[:, :, None]
    return ((w < lo) | (w > hi)).reshape(N, K)


def quantize_sqc(W16: np.ndarray, bits: np.ndarray, g: int = GROUP, lam: float = 0.1, n: int = 50):
    """Salience-Weighted Quantizer Calibration, function SQC of Algorithm 2, per (row, group).

    For every candidate tau: Delta = tau (w_max - w_min) / (2^b - 1), z = -round(tau w_min / Delta),
    fake-quantise the salient and the non-salient part of the group with the shared (Delta, z) and
    keep the candidate with the smallest L_s + L_us (first one on ties: the comparison is strict).
    Storage readings as in quantize_minmax: the range contains 0, Delta is rounded to fp16 before z,
    the codes and the losses are computed, a zero Delta becomes 1, z is clamped to [0, 2^b - 1].
    Losses are fp64 sums of squared errors taken in column order.

    Returns codes uint8 [N][K], scales fp16 [G][N], zeros fp16 [G][N], tau index int32 [G][N],
    loss fp64 [G][N] (= L_s + L_us of the chosen candidate), salient loss fp64 [G][N] (L_s of it).
    """
    N, K = W16.shape
    G = K // g
    assert K % g == 0 and len(bits) == G
    taus = sqc_tau_grid(lam, n)
    mask = salient_mask_3sigma(W16, g)
    codes = np.zeros((N, K), dtype=np.uint8)
    scales = np.zeros((G, N), dtype=np.float16)
    zeros = np.zeros((G, N), dtype=np.float16)
    tau_idx = np.zeros((G, N), dtype=np.int32)
    loss = np.zeros((G, N), dtype=np.float64)
    loss_s = np.zeros((G, N), dtype=np.float64)
    for j in range(G):
        b = int(bits[j])
        levels = float(2**b - 1)
        w = W16[:, j * g:(j + 1) * g].astype(np.float64)
        ms = mask[:, j * g:(j + 1) * g]
        lo = np.minimum(w.min(axis=1), 0.0)
        hi = np.maximum(w.max(axis=1), 0.0)
        best = np.full(N, np.inf)
        for ti, tau in enumerate(taus):
            with np.errstate(over="ignore"):
                s16 = (tau * (hi - lo) / levels).astype(np.float16)
            s16[np.isinf(s16)] = np.float16(65504.0)
            s16[s16 == 0] = np.float16(1.0)
            s = s16.astype(np.float64)
            z = np.clip(-np.rint(tau * lo / s), 0.0, levels) + 0.0
            q = np.clip(np.rint(w / s[:, None]) + z[:, None], 0.0, levels)
            err = w - s[:, None] * (q - z[:, None])
            sq = err * err
            L_s = np.zeros(N)
            L_us = np.zeros(N)
            for k in range(g):                       # column order, so that every implementation can follow it
                L_s = L_s + np.where(ms[:, k], sq[:, k], 0.0)
                L_us = L_us + np.where(ms[:, k], 0.0, sq[:, k])
            total = L_s + L_us
            take = total < best
            best = np.where(take, total, best)
            codes[take, j * g:(j + 1) * g] = q[take].astype(np.uint8)
            scales[j, take] = s16[take]
            zeros[j, take] = z[take].astype(np.float16)
            tau_idx[j, take] = ti
            loss[j, take] = total[take]
            loss_s[j, take] = L_s[take]
    return codes, scales, zeros, tau_idx, loss, loss_s


def quantize_sign_alpha_1bit(W16: np.ndarray, g: int = GROUP):
    """Eq. 2 for one-bit groups: w_b = sign(w) (sign(0) = +1), alpha = mean |w|.

    Expressed in the deployed (scale, zero, code) form: q = [w >= 0], z = 1/2,
    s = fp16(2 alpha), so that s (q - z) = +-alpha.  Returned with the layouts of
    quantize_minmax, every group at one bit.
    """
    N, K = W16.shape
    G = K // g
    w = W16.astype(np.float64).reshape(N, G, g)
    alpha = np.abs(w).mean(axis=2)
    codes = (w >= 0).astype(np.uint8).reshape(N, K)
    scales = (2.0 * alpha).astype(np.float16).T.copy()
    zeros = np.full((G, N), 0.5, dtype=np.float16)
    return codes, scales, zeros


def quantize_minmax_sign1(W16: np.ndarray, bits: np.ndarray, g: int = GROUP):
    """Eq. 1 for the groups of two or more bits, Eq. 2 (sign, alpha) for the one-bit groups: the
    quantizer the paper describes "when converted to 1-bit" (Sec. 3.1), in the deployed layouts."""
    bits = np.asarray(bits, dtype=np.uint8)
    codes, scales, zeros = quantize_minmax(W16, bits, g)
    c1, s1, z1 = quantize_sign_alpha_1bit(W16, g)
    for j in np.nonzero(bits == 1)[0]:
        codes[:, g * j:g * (j + 1)] = c1[:, g * j:g * (j + 1)]
        scales[j] = s1[j]
        zeros[j] = z1[j]
    return codes, scales, zeros


# --------------------------------------------------------------------------- dequantisation
def _expand_group_param(p: np.ndarray, g: int) -> np.ndarray:
    """[G][N] per-(group,row) parameter -> [N][K] per-element."""
    return np.repeat(np.asarray(p).T, g, axis=1)


def dequant_f64(codes, scales, zeros, g: int = GROUP) -> np.ndarray:
    """w-hat = s (q - z), exact in fp64 (the closed-form inverse inside Eq. 5)."""
    s = _expand_group_param(scales, g).astype(np.float64)
    z = _expand_group_param(zeros, g).astype(np.float64)
    return s * (codes.astype(np.float64) - z)


def dequant_f16(codes, scales, zeros, g: int = GROUP) -> np.ndarray:
    """fp16 materialisation: fp16_rn( f32(s) *_f32 ( f32(q) -_f32 f32(z) ) ).

    For integer or half-integer z both fp32 operations are exact, so this is the
    correctly rounded fp16 value of s (q - z).
    """
    s = _expand_group_param(scales, g).astype(np.float32)
    z = _expand_group_param(zeros, g).astype(np.float32)
    d = codes.astype(np.float32) - z
    with np.errstate(over="ignore"):
        return (s * d).astype(np.float16)


# --------------------------------------------------------------------------- linear layer
def linear_f64(x16, codes, scales, zeros, g: int = GROUP) -> np.ndarray:
    """y_ref = x @ W-hat^T with exact (unrounded) dequantised weights, fp64."""
    return x16.astype(np.float64) @ dequant_f64(codes, scales, zeros, g).T


def linear_rows_f64(x16, codes, scales, zeros, rows, g: int = GROUP) -> np.ndarray:
    """y_ref[:, rows] only (for sampled checks of large layers)."""
    rows = np.asarray(rows)
    return linear_f64(x16, codes[rows], np.asarray(scales)[:, rows], np.asarray(zeros)[:, rows], g)


# --------------------------------------------------------------------------- storage format
GROUP_SIZES = (32, 64, 128, 256, 512)


def ktile(g: int) -> int:
    """Columns of a K-tile of the packed format: the group itself up to 128 columns, else 128."""
    assert g in GROUP_SIZES
    return min(g, 128)


def ktile_bits(bits, g: int) -> np.ndarray:
    """Bit-width of every K-tile: a group of more than 128 columns is g/128 consecutive tiles of its width."""
    bits = np.asarray(bits, dtype=np.uint8)
    return np.repeat(bits, max(g // 128, 1))


def packed_bytes(N: int, K: int, bits, g: int = GROUP) -> int:
    """N*K*b-bar/8: groups are stored back to back without padding (App. B.2)."""
    assert K % g == 0 and len(bits) == K // g
    return g // 8 * N * int(np.asarray(bits, dtype=np.int64).sum())


def _item_bit_index(N, T, tile_prefix, b, t, unit, lane, half):
    """Bit offset, in the packed buffer, of bit 0 of one item (the T/4 bits a lane holds for one row).

    K-tile at byte (T/8)*N*B (B = bits of the K-tiles before it); inside it the 16-row tile t at t*2T*b; inside
    that the unit `unit` (2T bytes); inside that lane L at L*T/16 bytes; item `half` (0: even row, 1: odd row)
    at half*T/32 bytes.
    """
    byte = T // 8 * N * tile_prefix + t * 2 * T * b + 2 * T * unit
    return 8 * byte + (T // 2) * lane + (T // 4) * half


def pack(codes: np.ndarray, bits, g: int = GROUP) -> np.ndarray:
    """Pack codes [N][K] into the sliced bit-plane format; returns uint8 bytes.

    Format (N a multiple of 16, g in GROUP_SIZES).  K is cut into K-tiles of T = min(g, 128) columns; a group of
    more than 128 columns is g/128 consecutive K-tiles of its bit-width.  K-tiles are stored back to back; a tile
    of b bits takes N*T*b/8 bytes and holds, for each 16-row tile t, b units of 2T bytes.  The code is cut into
    slices (lo, w) listed in CODE_SLICES[b]; a slice of width w owns w consecutive units.  A unit is 32 lanes x
    T/16 bytes; lane L = 4*gq + c (gq = 0..7, c = 0..3) holds two little-endian items of T/4 bits, item 0 for row
    16t + 2gq and item 1 for row 16t + 2gq + 1.  Item (row r, slice (lo, w), unit u of the slice, c) has (T/4)/w
    fields; field f occupies bits [w f, w f + w) and stores slice (lo, w) of
    q[r, T jt + (T/4) c + ((T/4)/w) u + f]  (jt = index of the K-tile).  For g = 128 an item is a 32-bit word.
    """
    codes = np.asarray(codes, dtype=np.uint8)
    N, K = codes.shape
    assert g in GROUP_SIZES and K % g == 0 and N % 16 == 0 and len(bits) == K // g
    T = ktile(g)
    tb = ktile_bits(bits, g)
    n_bits = 8 * packed_bytes(N, K, bits, g)
    out_bits = np.zeros(n_bits, dtype=np.uint8)
    rows = np.arange(N)
    t, r = rows // 16, rows % 16
    gq, half = r // 2, r % 2
    prefix = 0
    for jt in range(K // T):
        b = int(tb[jt])
        q = codes[:, jt * T:(jt + 1) * T].astype(np.uint32)
        assert int(q.max(initial=0)) < 2**b, "code out of range for its group width"
        unit_base = 0
        for (lo, w) in CODE_SLICES[b]:
            nf = T // 4 // w
            for u in range(w):
                for c in range(4):
                    base = _item_bit_index(N, T, prefix, b, t, unit_base + u, 4 * gq + c, half)
                    for f in range(nf):
                        k = T // 4 * c + nf * u + f
                        v = (q[:, k] >> np.uint32(lo)) & np.uint32(2**w - 1)
                        for bit in range(w):
                            out_bits[base + w * f + bit] = (v >> np.uint32(bit)) & 1
            unit_base += w
        prefix += b
    return np.packbits(out_bits, bitorder="little")


def unpack(packed: np.ndarray, N: int, K: int, bits, g: int = GROUP) -> np.ndarray:
    """Inverse of pack: bytes -> codes uint8 [N][K]."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    assert packed.size == packed_bytes(N, K, bits, g)
    in_bits = np.unpackbits(packed, bitorder="little")
    T = ktile(g)
    tb = ktile_bits(bits, g)
    codes = np.zeros((N, K), dtype=np.uint8)
    rows = np.arange(N)
    t, r = rows // 16, rows % 16
    gq, half = r // 2, r % 2
    prefix = 0
    for jt in range(K // T):
        b = int(tb[jt])
        unit_base = 0
        for (lo, w) in CODE_SLICES[b]:
            nf = T // 4 // w
            for u in range(w):
                for c in range(4):
                    base = _item_bit_index(N, T, prefix, b, t, unit_base + u, 4 * gq + c, half)
                    for f in range(nf):
                        k = jt * T + T // 4 * c + nf * u + f
                        for bit in range(w):
                            codes[:, k] |= (in_bits[base + w * f + bit] << (lo + bit)).astype(np.uint8)
            unit_base += w
        prefix += b
    return codes


# --------------------------------------------------------------------------- SBA search (Algorithm 2, func SBA)
def softmax_kl(y_ref: np.ndarray, y_q: np.ndarray) -> np.ndarray:
    """D_kl( softmax(y_ref[t]) || softmax(y_q[t]) ) for every token row t, natural logarithm.

    The objective of Eq. 4 compares the layer outputs x w^T and x w-hat^T; the appendix on the
    evaluation function of SBA turns each output into a probability distribution with a softmax
    first.  The softmax runs over the output features of one token; one value per token is
    returned.  Written as the definition: p = exp(y - logsumexp(y)), sum_n p_n (log p_n - log q_n).
    """
    a = np.asarray(y_ref, dtype=np.float64)
    b = np.asarray(y_q, dtype=np.float64)
    out = np.empty(a.shape[0], dtype=np.float64)
    for t in range(a.shape[0]):
        la = a[t] - a[t].max()
        lb = b[t] - b[t].max()
        log_p = la - np.log(np.exp(la).sum())
        log_q = lb - np.log(np.exp(lb).sum())
        out[t] = float((np.exp(log_p) * (log_p - log_q)).sum())
    return out


def sba_search(W16: np.ndarray, x16: np.ndarray, act_norm: np.ndarray, avg_bits: int, g: int = GROUP,
               include_uniform: bool = True):
    """Salience-Determined Bit Allocation, func SBA of Algorithm 2 (Sec. 3.2.2, Eq. 4).

    Groups are ranked by salience; for p = 0 (uniform; the loop of Algorithm 2 starts at 1, the
    appendix on the search names the uniform map as one end of the range), 1, ..., floor(G/2) the p
    most salient groups get N-bar+1 bits and the p least salient N-bar-1 (the double pointer), the
    weight is fake-quantised with the quantizer of Eq. 1 under that map, and the candidate's error
    is the KL divergence between the softmax of the full-precision output x w^T and of x w-hat^T,
    averaged over the calibration tokens.  The first p with the smallest error wins (Algorithm 2
    compares with '<').  Returns (p_star, bits[G], errors[list over the candidates p]).
    """
    W = W16.astype(np.float64)
    x = x16.astype(np.float64)
    S = group_salience(W16, act_norm, g)
    G = S.shape[0]
    y_f = x @ W.T
    first = 0 if include_uniform else 1
    errors = []
    for p in range(first, G // 2 + 1):
        bits = allocate_bits(S, avg_bits, p)
        codes, scales, zeros = quantize_minmax(W16, bits, g)
        y_q = linear_f64(x16, codes, scales, zeros, g)
        errors.append(float(softmax_kl(y_f, y_q).mean()))
    best = 0
    for i in range(1, len(errors)):
        if errors[i] < errors[best]:
            best = i
    p_star = first + best
    return p_star, allocate_bits(S, avg_bits, p_star), errors


# --------------------------------------------------------------------------- GPTQ error compensation
def gptq_hessian(x16: np.ndarray) -> np.ndarray:
    """H = (1/P) sum_k x_k x_k^T over the P calibration tokens (Algorithm 1, first step), fp64 [K][K]."""
    x = x16.astype(np.float64)
    return x.T @ x / x.shape[0]


def gptq_factor(H: np.ndarray, lam: float = 0.01):
    """H_in = Cholesky((H + lambda I)^-1) (Algorithm 1, second step): the upper-triangular U with
    U^T U = (H + lambda I)^-1.  Returns (U, dead).

    Readings: lambda is relative to the mean diagonal of H (lambda_abs = lam * mean(diag H), the
    convention of the GPTQ backbone the paper builds on), so the scale of H (the 1/P) does not matter;
    an input channel that is zero in every token (`dead`) gets H_kk = 1 before damping and its weight
    column is treated as zero by the caller.
    """
    import scipy.linalg
    H = H.copy()
    dead = np.diag(H) == 0
    H[dead, dead] = 1.0
    K = H.shape[0]
    Hd = H + lam * np.mean(np.diag(H)) * np.eye(K)
    U = scipy.linalg.cholesky(np.linalg.inv(Hd), lower=False)
    return U, dead


def gptq_quantize(W16: np.ndarray, x16: np.ndarray, bits, lam: float = 0.01, quantizer: str = "sqc", g: int = GROUP):
    """Main loop of Algorithm 1 with a given bit map: group by group, quantise the CURRENT weights of
    the group with SQC (or plain Eq. 1), then push the group's error onto the columns not yet
    quantised:  E = (w_b - w-hat_b) / H_in[b, b]  (right division by the diagonal block),
                w[:, after] -= E @ H_in[b, after].

    Readings: the running weights are kept in fp64; the quantizer is given the group rounded to fp16
    (its input type: the paper's weights are FP16) and returns fp16 scale and zero point, and the
    error is taken against the exact s (q - z).  Returns (codes, scales, zeros, w_running) with the
    layouts of quantize_minmax; w_running is the fp64 matrix after the last update.
    """
    bits = np.asarray(bits)
    N, K = W16.shape
    G = K // g
    U, dead = gptq_factor(gptq_hessian(x16), lam)
    w = W16.astype(np.float64).copy()
    w[:, dead] = 0.0
    codes = np.zeros((N, K), dtype=np.uint8)
    scales = np.zeros((G, N), dtype=np.float16)
    zeros = np.zeros((G, N), dtype=np.float16)
    for j in range(G):
        cols = slice(g * j, g * (j + 1))
        wb16 = w[:, cols].astype(np.float16)
        if quantizer == "sqc":
            q, s, z = quantize_sqc(wb16, bits[j:j + 1], g)[:3]
        elif quantizer == "minmax":
            q, s, z = quantize_minmax(wb16, bits[j:j + 1], g)
        else:
            raise ValueError(quantizer)
        codes[:, cols], scales[j], zeros[j] = q, s[0], z[0]
        w_hat = s[0].astype(np.float64)[:, None] * (q.astype(np.float64) - z[0].astype(np.float64)[:, None])
        delta = w[:, cols] - w_hat
        # E U_bb = delta  (U_bb upper triangular)
        E = np.linalg.solve(U[cols, cols].T, delta.T).T
        w[:, g * (j + 1):] -= E @ U[cols, g * (j + 1):]
    return codes, scales, zeros, w


def gptq_proxy_loss(W16: np.ndarray, W_hat: np.ndarray, x16: np.ndarray) -> float:
    """|| (w - w-hat) x^T ||_F^2 / P: the layer-output error the compensation minimises."""
    d = (W16.astype(np.float64) - W_hat) @ x16.astype(np.float64).T
    return float((d * d).sum() / x16.shape[0])


# --------------------------------------------------------------------------- convenience
def make_layer(W16, act_norm, avg_bits: int, g: int = GROUP, p: int | None = None):
    """Salience -> bit map -> quantizer, the pipeline of the benchmark configs."""
    bits = allocate_bits(group_salience(W16, act_norm, g), avg_bits, p)
    codes, scales, zeros = quantize_minmax(W16, bits, g)
    return bits, codes, scales, zeros
