// GPTQ error compensation around the group quantizer (Algorithm 1), sm_100a, fp64 throughout.
//
//   H     = (1/P) sum_k x_k x_k^T                       gptq_hessian_kernel (upper tiles only)
//   H    += lambda mean(diag H) I, dead channels         gptq_damp_kernel
//   H     = R R^T, R upper triangular                    gptq_chol_{diag,panel,trail}_kernel, last block first
//   U     = R^-1  (so U^T U = (H + lambda I)^-1: the Cholesky factor Algorithm 1 calls H_in)
//                                                        diagonal blocks with the factor, then gptq_inv_pair{1,2}_kernel (doubling)
//   per group b:  quantise fp16(w_b) with SQC or Eq. 1 (the library's quantizer kernels),
//                 E = (w_b - w-hat_b) R_bb                gptq_error_kernel  (R_bb = U_bb^-1: no solve)
//                 w[:, after] -= E U[b, after]            gptq_update_kernel
//
// Everything is a fixed-order fp64 sum, so a layer gives the same codes on every run.  The 64 x 64 x 16
// register-tiled product below serves the four GEMM-shaped steps; the sequential parts (the factor of
// a diagonal block, the triangular solves against it) run one thread per row or column.
#include "slim_common.cuh"

namespace slim {

constexpr int kFB = 64;            // block of the factorisation
constexpr int kFK = 16;            // depth of one shared-memory stage of the tile product
constexpr int kFPad = kFB + 2;    // row stride of the staged operands: even, so that pairs of doubles stay 16-byte aligned

// ------------------------------------------------------------------------------------------ 64 x 64 tile product
// acc[a][b] (rows tidx(ty, a), columns tidx(tx, b) of the tile) += sum_k A(i, k) B(k, j); the operands of
// one stage are put into As[k][i], Bs[k][j] by the two fill functors (called by all 256 threads with the
// stage's first k), zero where the operand does not exist.  A thread owns the index pairs (2t, 2t + 1) and
// (32 + 2t, 33 + 2t), so that the 16 threads of a row read consecutive 16-byte pieces of shared memory.
__device__ __forceinline__ int tidx(int t, int e) { return 2 * t + (e & 1) + 32 * (e >> 1); }
// An operand gives load(k0, r): the thread's four elements of the stage that starts at k0, from global
// memory, and store(S, r): their places in the staged array.  The next stage is loaded into registers
// while the current one is multiplied.
template <class OpA, class OpB>
__device__ __forceinline__ void tile_mac(double (&acc)[4][4], int klen, const OpA& opa, const OpB& opb,
                                         double (*As)[kFPad], double (*Bs)[kFPad]) {
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    double ra[4], rb[4];
    opa.load(0, ra);
    opb.load(0, rb);
    for (int k0 = 0; k0 < klen; k0 += kFK) {
        OpA::store(As, ra);
        OpB::store(Bs, rb);
        __syncthreads();
        if (k0 + kFK < klen) {
            opa.load(k0 + kFK, ra);
            opb.load(k0 + kFK, rb);
        }
#pragma unroll
        for (int k = 0; k < kFK; ++k) {
            const double2 a01 = *reinterpret_cast<const double2*>(&As[k][2 * ty]), a23 = *reinterpret_cast<const double2*>(&As[k][32 + 2 * ty]);
            const double2 b01 = *reinterpret_cast<const double2*>(&Bs[k][2 * tx]), b23 = *reinterpret_cast<const double2*>(&Bs[k][32 + 2 * tx]);
            const double a[4] = {a01.x, a01.y, a23.x, a23.y}, b[4] = {b01.x, b01.y, b23.x, b23.y};
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int f = 0; f < 4; ++f) acc[e][f] = fma(a[e], b[f], acc[e][f]);
        }
        __syncthreads();
    }
}
// Operand stored with the tile index contiguous: element (k, i) = src[k * ld + i], k < kmax, i < imax.
struct OpK {
    const double* src; size_t ld; int kmax; int imax = 1 << 30;
    __device__ __forceinline__ void load(int k0, double (&r)[4]) const {
        const int k = k0 + (threadIdx.x >> 4), i = (threadIdx.x & 15) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) r[e] = (k < kmax && i + e < imax) ? src[static_cast<size_t>(k) * ld + i + e] : 0.0;
    }
    __device__ __forceinline__ static void store(double (*S)[kFPad], const double (&r)[4]) {
        const int k = threadIdx.x >> 4, i = (threadIdx.x & 15) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) S[k][i + e] = r[e];
    }
};
struct OpKHalf {
    const __half* src; size_t ld; int kmax;
    __device__ __forceinline__ void load(int k0, double (&r)[4]) const {
        const int k = k0 + (threadIdx.x >> 4), i = (threadIdx.x & 15) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) r[e] = k < kmax ? static_cast<double>(__half2float(src[static_cast<size_t>(k) * ld + i + e])) : 0.0;
    }
    __device__ __forceinline__ static void store(double (*S)[kFPad], const double (&r)[4]) { OpK::store(S, r); }
};
// Operand stored with k contiguous: element (i, k) = src[i * ld + k], k < kmax; rows i >= imax do not exist.
struct OpI {
    const double* src; size_t ld; int kmax, imax;
    __device__ __forceinline__ void load(int k0, double (&r)[4]) const {
        const int i = threadIdx.x >> 2, k = k0 + (threadIdx.x & 3) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) r[e] = (k + e < kmax && i < imax) ? src[static_cast<size_t>(i) * ld + k + e] : 0.0;
    }
    __device__ __forceinline__ static void store(double (*S)[kFPad], const double (&r)[4]) {
        const int i = threadIdx.x >> 2, k = (threadIdx.x & 3) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) S[k + e][i] = r[e];
    }
};

// ------------------------------------------------------------------------------------------ Hessian
// H[i][j] = (1/T) sum_t x[t][i] x[t][j] for the tiles on and above the diagonal (t ascending).
__global__ void __launch_bounds__(256) gptq_hessian_kernel(const __half* __restrict__ x, double* __restrict__ H, int T, int K) {
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (bj < bi) return;
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    double acc[4][4] = {};
    tile_mac(acc, T, OpKHalf{x + kFB * bi, static_cast<size_t>(K), T}, OpKHalf{x + kFB * bj, static_cast<size_t>(K), T}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const double inv = 1.0 / static_cast<double>(T);
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f)
            H[static_cast<size_t>(kFB * bi + tidx(ty, e)) * K + kFB * bj + tidx(tx, f)] = acc[e][f] * inv;
}

// dead[k] = (H_kk == 0); such a channel gets H_kk = 1; then H_kk += lambda * mean(diag H).  One CTA.
__global__ void __launch_bounds__(1024) gptq_damp_kernel(double* __restrict__ H, uint8_t* __restrict__ dead, int K, double lambda) {
    __shared__ double part[1024];
    double s = 0.0;
    for (int k = threadIdx.x; k < K; k += 1024) {
        double d = H[static_cast<size_t>(k) * K + k];
        const bool z = d == 0.0;
        dead[k] = z ? 1 : 0;
        if (z) { d = 1.0; H[static_cast<size_t>(k) * K + k] = 1.0; }
        s += d;
    }
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    const double add = lambda * (part[0] / static_cast<double>(K));
    for (int k = threadIdx.x; k < K; k += 1024) H[static_cast<size_t>(k) * K + k] += add;
}

// ------------------------------------------------------------------------------------------ H = R R^T, R upper
// Diagonal block at b0: the unblocked recursion from the last column to the first,
//   R_cc = sqrt(S_cc),  R_ic = S_ic / R_cc (i < c),  S_ij -= R_ic R_jc (i <= j < c),   in place;
// then its inverse (thread j: column j by back substitution, u_i = (delta_ij - sum_{l > i} R_il u_l) / R_ii,
// held in registers), which is the diagonal block of U and turns the panel solve into a product.
__global__ void __launch_bounds__(256) gptq_chol_diag_kernel(double* __restrict__ A, double* __restrict__ U, int K, int b0) {
    __shared__ double S[kFB][kFB + 1];
    double* blk = A + static_cast<size_t>(b0) * K + b0;
    for (int e = threadIdx.x; e < kFB * kFB; e += 256) {
        const int i = e >> 6, j = e & 63;
        S[i][j] = j >= i ? blk[static_cast<size_t>(i) * K + j] : 0.0;
    }
    __syncthreads();
    // the factor runs on registers: thread (ty, tx) owns rows ty + 16 a, columns tx + 16 b
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    __shared__ double col[kFB], diag;
    double r[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) r[a][b] = S[ty + 16 * a][tx + 16 * b];
    for (int c = kFB - 1; c >= 0; --c) {
        const int cs = c >> 4, cl = c & 15;
        if (ty == cl && tx == cl) {
            double v = 0.0;
#pragma unroll
            for (int a = 0; a < 4; ++a)
                if (a == cs) v = r[a][a];
            diag = sqrt(v);
        }
        __syncthreads();
        const double d = diag;
        if (tx == cl) {
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int i = ty + 16 * a;
                double v = 0.0;
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (b == cs) v = r[a][b];
                v = i < c ? v / d : (i == c ? d : v);
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (b == cs) r[a][b] = v;
                col[i] = v;
            }
        }
        __syncthreads();
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = ty + 16 * a, j = tx + 16 * b;
                if (j < c && i <= j) r[a][b] -= col[i] * col[j];
            }
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) S[ty + 16 * a][tx + 16 * b] = r[a][b];
    __syncthreads();
    for (int e = threadIdx.x; e < kFB * kFB; e += 256) {
        const int i = e >> 6, j = e & 63;
        if (j >= i) blk[static_cast<size_t>(i) * K + j] = S[i][j];
    }
    // The inverse, in place in S.  16 x 16 diagonal blocks by back substitution (thread = one column,
    // u_i = (delta_ij - sum_{l > i} R_il u_l) / R_ii, in registers); then two doubling levels: for neighbouring
    // segments A, C with known inverses the block above C becomes -A^-1 (B C^-1).  The lower triangle of S is
    // zero, so the sums run over whole segments.
    __shared__ double Tm[32][33];
    {
        const int o = threadIdx.x & 48, jl = threadIdx.x & 15;      // threads 0..63: column jl of the block at o
        double u[16];
        if (threadIdx.x < kFB) {
#pragma unroll
            for (int i = 15; i >= 0; --i) {
                double v = i == jl ? 1.0 : 0.0;                    // rows below the column's own stay zero
#pragma unroll
                for (int l = i + 1; l < 16; ++l) v = fma(-S[o + i][o + l], u[l], v);
                u[i] = v / S[o + i][o + i];
            }
        }
        __syncthreads();                                           // every column has read R before any is replaced
        if (threadIdx.x < kFB) {
#pragma unroll
            for (int i = 0; i < 16; ++i) S[o + i][o + jl] = u[i];
        }
        __syncthreads();
    }
    for (int seg = 16; seg < kFB; seg *= 2) {
        // T = B C^-1 for every pair of segments: pair at o = 2 seg p, B = S[o .. o+seg)[o+seg .. o+2seg)
        const int per_pair = seg * seg, n_out = per_pair * (kFB / (2 * seg));
        for (int e = threadIdx.x; e < n_out; e += 256) {
            const int pr = e / per_pair, q = e - pr * per_pair, i = q / seg, j = q - i * seg, o = 2 * seg * pr;
            double v = 0.0;
            for (int k = 0; k < seg; ++k) v = fma(S[o + i][o + seg + k], S[o + seg + k][o + seg + j], v);
            Tm[(seg == 16 ? 16 * pr : 0) + i][j] = v;
        }
        __syncthreads();
        for (int e = threadIdx.x; e < n_out; e += 256) {
            const int pr = e / per_pair, q = e - pr * per_pair, i = q / seg, j = q - i * seg, o = 2 * seg * pr;
            double v = 0.0;
            for (int k = 0; k < seg; ++k) v = fma(S[o + i][o + k], Tm[(seg == 16 ? 16 * pr : 0) + k][j], v);
            S[o + i][o + seg + j] = -v;
        }
        __syncthreads();
    }
    double* ub = U + static_cast<size_t>(b0) * K + b0;
    for (int e = threadIdx.x; e < kFB * kFB; e += 256) ub[static_cast<size_t>(e >> 6) * K + (e & 63)] = S[e >> 6][e & 63];
}

// Panel above the diagonal block: X R_bb^T = A[I, b], i.e. X = A[I, b] (R_bb^-1)^T, one 64 x 64 tile per CTA, in place.
__global__ void __launch_bounds__(256) gptq_chol_panel_kernel(double* __restrict__ A, const double* __restrict__ U, int K, int b0) {
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    double* pan = A + static_cast<size_t>(kFB) * blockIdx.x * K + b0;
    const double* rinv = U + static_cast<size_t>(b0) * K + b0;
    double acc[4][4] = {};
    tile_mac(acc, kFB, OpI{pan, static_cast<size_t>(K), kFB, kFB}, OpI{rinv, static_cast<size_t>(K), kFB, kFB}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) pan[static_cast<size_t>(tidx(ty, e)) * K + tidx(tx, f)] = acc[e][f];
}

// Trailing update: A[I, J] -= R[I, b] R[J, b]^T for the tiles I <= J in front of block b.
__global__ void __launch_bounds__(256) gptq_chol_trail_kernel(double* __restrict__ A, int K, int b0) {
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (bj < bi) return;
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    double acc[4][4] = {};
    const double* pi = A + static_cast<size_t>(kFB) * bi * K + b0;
    const double* pj = A + static_cast<size_t>(kFB) * bj * K + b0;
    tile_mac(acc, kFB, OpI{pi, static_cast<size_t>(K), kFB, kFB}, OpI{pj, static_cast<size_t>(K), kFB, kFB}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f)
            A[static_cast<size_t>(kFB * bi + tidx(ty, e)) * K + kFB * bj + tidx(tx, f)] -= acc[e][f];
}

// ------------------------------------------------------------------------------------------ U = R^-1
// Off-diagonal blocks by doubling: with the inverses of two neighbouring diagonal segments A (s x s at o) and
// C (s2 x s2 at o + s) known, the block above C is  -A^-1 (B C^-1),  B = R[A rows, C columns].
// First half: T = B C^-1, left in the unused mirror block U[C rows, A columns] (column tile j of the upper
// triangular C^-1 has its nonzeros in k < 64 (j + 1)).
__global__ void __launch_bounds__(256) gptq_inv_pair1_kernel(const double* R, double* U, int K, int s) {
    const int o = 2 * s * blockIdx.z, s2 = min(s, K - o - s);
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (s2 <= 0 || kFB * tj >= s2) return;
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    double acc[4][4] = {};
    const double* a = R + static_cast<size_t>(o + kFB * ti) * K + o + s;                 // B[i][k]
    const double* b = U + static_cast<size_t>(o + s) * K + o + s + kFB * tj;             // C^-1[k][j]
    const int klen = kFB * (tj + 1);
    tile_mac(acc, klen, OpI{a, static_cast<size_t>(K), klen, kFB}, OpK{b, static_cast<size_t>(K), klen}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    double* t = U + static_cast<size_t>(o + s + kFB * tj) * K + o + kFB * ti;            // T stored transposed: T^T[j][i]
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) t[static_cast<size_t>(tidx(tx, f)) * K + tidx(ty, e)] = acc[e][f];
}
// Second half: U[A rows, C columns] = -A^-1 T (row tile i of the upper triangular A^-1 has its nonzeros in k >= 64 i).
__global__ void __launch_bounds__(256) gptq_inv_pair2_kernel(double* U, int K, int s) {
    const int o = 2 * s * blockIdx.z, s2 = min(s, K - o - s);
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (s2 <= 0 || kFB * tj >= s2) return;
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    double acc[4][4] = {};
    const int kbeg = kFB * ti, klen = s - kbeg;
    const double* a = U + static_cast<size_t>(o + kFB * ti) * K + o + kbeg;              // A^-1[i][k], k from kbeg
    const double* b = U + static_cast<size_t>(o + s + kFB * tj) * K + o + kbeg;          // T^T[j][k]
    tile_mac(acc, klen, OpI{a, static_cast<size_t>(K), klen, kFB}, OpI{b, static_cast<size_t>(K), klen, kFB}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    double* out = U + static_cast<size_t>(o + kFB * ti) * K + o + s + kFB * tj;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) out[static_cast<size_t>(tidx(ty, e)) * K + tidx(tx, f)] = -acc[e][f];
}
// The mirror blocks held T: the lower triangle goes back to zero.
__global__ void __launch_bounds__(256) gptq_zero_lower_kernel(double* U, int K) {
    const int i = blockIdx.y, j0 = blockIdx.x * 256 + threadIdx.x;
    if (j0 < i) U[static_cast<size_t>(i) * K + j0] = 0.0;
}

// ------------------------------------------------------------------------------------------ the loop over the groups
// Running weights: w = fp64(W), dead input channels zeroed.
__global__ void __launch_bounds__(256) gptq_init_kernel(const __half* __restrict__ W, const uint8_t* __restrict__ dead,
                                                        double* __restrict__ w, size_t total, int K) {
    const size_t i = static_cast<size_t>(blockIdx.x) * 256 + threadIdx.x;
    if (i >= total) return;
    const int k = static_cast<int>(i % static_cast<size_t>(K));
    w[i] = dead[k] ? 0.0 : static_cast<double>(__half2float(W[i]));
}
// The group's current weights rounded to fp16 (one rounding), [N][g]: the quantizer's input.
__global__ void __launch_bounds__(256) gptq_round_kernel(const double* __restrict__ w, __half* __restrict__ wb, int N, int K, int c0, int g) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= N * g) return;
    const int n = i / g, c = i - n * g;
    wb[i] = __double2half(w[static_cast<size_t>(n) * K + c0 + c]);
}
// delta = w_b - s (q - z) for ROWS rows per CTA, codes copied into the layer's array,
// E[n][c] = sum_{c' <= c} delta[n][c'] R[c0 + c'][c0 + c]   (thread c of the group's GS columns, c' ascending).
template <int GS, int ROWS>
__global__ void __launch_bounds__(GS) gptq_error_kernel(const double* __restrict__ w, const uint8_t* __restrict__ qb,
                                                        const __half* __restrict__ s_row, const __half* __restrict__ z_row,
                                                        const double* __restrict__ R, uint8_t* __restrict__ codes,
                                                        double* __restrict__ E, int N, int K, int c0) {
    __shared__ double delta[ROWS][GS];
    const int c = threadIdx.x, n0 = ROWS * blockIdx.x;
    for (int r = 0; r < ROWS; ++r) {
        const int n = n0 + r;
        double d = 0.0;
        if (n < N) {
            const uint8_t q = qb[static_cast<size_t>(n) * GS + c];
            codes[static_cast<size_t>(n) * K + c0 + c] = q;
            const double sc = static_cast<double>(__half2float(s_row[n])), zp = static_cast<double>(__half2float(z_row[n]));
            d = w[static_cast<size_t>(n) * K + c0 + c] - sc * (static_cast<double>(q) - zp);
        }
        delta[r][c] = d;
    }
    __syncthreads();
    double acc[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) acc[r] = 0.0;
    for (int c2 = 0; c2 <= c; ++c2) {
        const double rv = R[static_cast<size_t>(c0 + c2) * K + c0 + c];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) acc[r] = fma(delta[r][c2], rv, acc[r]);
    }
    for (int r = 0; r < ROWS; ++r)
        if (n0 + r < N) E[static_cast<size_t>(n0 + r) * GS + c] = acc[r];
}
// w[n][k] -= sum_c E[n][c] U[c0 + c][k] for the columns k >= k0 = c0 + g (c ascending).
__global__ void __launch_bounds__(256) gptq_update_kernel(double* __restrict__ w, const double* __restrict__ E,
                                                          const double* __restrict__ U, int N, int K, int c0, int g) {
    __shared__ __align__(16) double As[kFK][kFPad], Bs[kFK][kFPad];
    const int n0 = kFB * blockIdx.y, k0 = c0 + g + kFB * blockIdx.x;
    double acc[4][4] = {};
    tile_mac(acc, g, OpI{E + static_cast<size_t>(n0) * g, static_cast<size_t>(g), g, N - n0},
             OpK{U + static_cast<size_t>(c0) * K + k0, static_cast<size_t>(K), g, K - k0}, As, Bs);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int n = n0 + tidx(ty, e);
        if (n >= N) continue;
#pragma unroll
        for (int f = 0; f < 4; ++f) {
            const int k = k0 + tidx(tx, f);
            if (k < K) w[static_cast<size_t>(n) * K + k] -= acc[e][f];      // groups of 32 columns end in the middle of a tile
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
struct GptqLayout {
    size_t dead, R, U, w, E, wb, qb, total;
};
static size_t up256(size_t v) { return (v + 255) / 256 * 256; }
static int gptq_layout(int T, int N, int K, int g, GptqLayout* lay) {
    if (lay == nullptr || T < 1 || N < 0 || K < 1) return SLIM_ERR_INVALID_ARG;
    if (g != 32 && g != 64 && g != 128 && g != 256 && g != 512) return SLIM_ERR_UNSUPPORTED;
    if (K % g != 0 || K % SLIM_GROUP != 0 || K / SLIM_GROUP > SLIM_MAX_GROUPS) return SLIM_ERR_UNSUPPORTED;
    size_t off = 0;
    lay->dead = off; off += up256(static_cast<size_t>(K));
    lay->R = off; off += up256(static_cast<size_t>(K) * K * sizeof(double));
    lay->U = off; off += up256(static_cast<size_t>(K) * K * sizeof(double));
    lay->w = off; off += up256(static_cast<size_t>(N) * K * sizeof(double));
    lay->E = off; off += up256(static_cast<size_t>(N) * g * sizeof(double));
    lay->wb = off; off += up256(static_cast<size_t>(N) * g * sizeof(__half));
    lay->qb = off; off += up256(static_cast<size_t>(N) * g);
    lay->total = off;
    return SLIM_OK;
}

// x -> U (and the dead-channel flags) inside the workspace.
static int gptq_factor_into(const void* x, int T, int K, double lambda, uint8_t* ws, const GptqLayout& lay, cudaStream_t s) {
    double* R = reinterpret_cast<double*>(ws + lay.R);
    double* U = reinterpret_cast<double*>(ws + lay.U);
    uint8_t* dead = ws + lay.dead;
    const int nb = K / kFB;
    gptq_hessian_kernel<<<dim3(nb, nb), 256, 0, s>>>(static_cast<const __half*>(x), R, T, K);
    gptq_damp_kernel<<<1, 1024, 0, s>>>(R, dead, K, lambda);
    SLIM_CUDA_TRY(cudaMemsetAsync(U, 0, static_cast<size_t>(K) * K * sizeof(double), s));
    for (int b = nb - 1; b >= 0; --b) {
        gptq_chol_diag_kernel<<<1, 256, 0, s>>>(R, U, K, kFB * b);
        if (b > 0) {
            gptq_chol_panel_kernel<<<b, 256, 0, s>>>(R, U, K, kFB * b);
            gptq_chol_trail_kernel<<<dim3(b, b), 256, 0, s>>>(R, K, kFB * b);
        }
    }
    SLIM_CUDA_TRY(cudaGetLastError());
    for (int seg = kFB; seg < K; seg *= 2) {
        const dim3 grid(seg / kFB, seg / kFB, (K + 2 * seg - 1) / (2 * seg));
        gptq_inv_pair1_kernel<<<grid, 256, 0, s>>>(R, U, K, seg);
        gptq_inv_pair2_kernel<<<grid, 256, 0, s>>>(U, K, seg);
    }
    gptq_zero_lower_kernel<<<dim3((K + 255) / 256, K), 256, 0, s>>>(U, K);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

extern "C" {

int slim_gptq_workspace_bytes(int T, int N, int K, int g, size_t* out_bytes) {
    if (out_bytes == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::GptqLayout lay;
    const int st = slim::gptq_layout(T, N, K, g, &lay);
    if (st != SLIM_OK) return st;
    *out_bytes = lay.total;
    return SLIM_OK;
}

int slim_gptq_factor(const void* x, int T, int K, double lambda, double* U_out, uint8_t* dead_out,
                     void* workspace, size_t workspace_bytes, void* stream) {
    slim::GptqLayout lay;
    const int st = slim::gptq_layout(T, 0, K, SLIM_GROUP, &lay);
    if (st != SLIM_OK) return st;
    if (!(lambda > 0.0) || x == nullptr || U_out == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(x) || !slim::aligned16(U_out)) return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < lay.total) return SLIM_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SLIM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int st2 = slim::gptq_factor_into(x, T, K, lambda, ws, lay, s);
    if (st2 != SLIM_OK) return st2;
    SLIM_CUDA_TRY(cudaMemcpyAsync(U_out, ws + lay.U, static_cast<size_t>(K) * K * sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (dead_out != nullptr) SLIM_CUDA_TRY(cudaMemcpyAsync(dead_out, ws + lay.dead, static_cast<size_t>(K), cudaMemcpyDeviceToDevice, s));
    return SLIM_OK;
}

int slim_gptq_quantize(const void* W, const void* x, const uint8_t* bits_host, double lambda, int use_sqc,
                       uint8_t* codes, void* scales, void* zeros, double* w_running,
                       int N, int K, int T, int g, void* workspace, size_t workspace_bytes, void* stream) {
    slim::GptqLayout lay;
    int st = slim::gptq_layout(T, N, K, g, &lay);
    if (st != SLIM_OK) return st;
    if (bits_host == nullptr || N % 16 != 0) return bits_host == nullptr ? SLIM_ERR_INVALID_ARG : SLIM_ERR_UNSUPPORTED;
    const int G = K / g;
    for (int j = 0; j < G; ++j)
        if (bits_host[j] < 1 || bits_host[j] > 4) return SLIM_ERR_INVALID_ARG;
    if (!(lambda > 0.0)) return SLIM_ERR_INVALID_ARG;
    if (N == 0) return SLIM_OK;
    if (W == nullptr || x == nullptr || codes == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(W) || !slim::aligned16(x) || !slim::aligned16(codes) || !slim::aligned16(scales) || !slim::aligned16(zeros))
        return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < lay.total) return SLIM_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SLIM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    st = slim::gptq_factor_into(x, T, K, lambda, ws, lay, s);
    if (st != SLIM_OK) return st;

    const double* R = reinterpret_cast<const double*>(ws + lay.R);
    const double* U = reinterpret_cast<const double*>(ws + lay.U);
    double* w = reinterpret_cast<double*>(ws + lay.w);
    double* E = reinterpret_cast<double*>(ws + lay.E);
    __half* wb = reinterpret_cast<__half*>(ws + lay.wb);
    uint8_t* qb = ws + lay.qb;
    __half* sc = static_cast<__half*>(scales);
    __half* zp = static_cast<__half*>(zeros);
    const size_t total = static_cast<size_t>(N) * K;
    slim::gptq_init_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, s>>>(static_cast<const __half*>(W), ws + lay.dead, w, total, K);
    SLIM_CUDA_TRY(cudaGetLastError());
    for (int j = 0; j < G; ++j) {
        const int c0 = g * j;
        slim::gptq_round_kernel<<<(N * g + 255) / 256, 256, 0, s>>>(w, wb, N, K, c0, g);
        SLIM_CUDA_TRY(cudaGetLastError());
        const uint8_t b1[1] = {bits_host[j]};
        // the group as a one-group layer of g columns
        st = use_sqc ? slim_quantize_sqc(wb, b1, qb, sc + static_cast<size_t>(j) * N, zp + static_cast<size_t>(j) * N, nullptr,
                                         N, g, g, 0.1, 50, stream)
                     : slim_quantize_minmax(wb, b1, qb, sc + static_cast<size_t>(j) * N, zp + static_cast<size_t>(j) * N,
                                            N, g, g, stream);
        if (st != SLIM_OK) return st;
        const __half* s_row = sc + static_cast<size_t>(j) * N;
        const __half* z_row = zp + static_cast<size_t>(j) * N;
        switch (g) {
            case 32: slim::gptq_error_kernel<32, 16><<<(N + 15) / 16, 32, 0, s>>>(w, qb, s_row, z_row, R, codes, E, N, K, c0); break;
            case 64: slim::gptq_error_kernel<64, 16><<<(N + 15) / 16, 64, 0, s>>>(w, qb, s_row, z_row, R, codes, E, N, K, c0); break;
            case 128: slim::gptq_error_kernel<128, 16><<<(N + 15) / 16, 128, 0, s>>>(w, qb, s_row, z_row, R, codes, E, N, K, c0); break;
            case 256: slim::gptq_error_kernel<256, 16><<<(N + 15) / 16, 256, 0, s>>>(w, qb, s_row, z_row, R, codes, E, N, K, c0); break;
            default: slim::gptq_error_kernel<512, 8><<<(N + 7) / 8, 512, 0, s>>>(w, qb, s_row, z_row, R, codes, E, N, K, c0); break;
        }
        if (j + 1 < G)
            slim::gptq_update_kernel<<<dim3((K - c0 - g + slim::kFB - 1) / slim::kFB, (N + slim::kFB - 1) / slim::kFB), 256, 0, s>>>(w, E, U, N, K, c0, g);
        SLIM_CUDA_TRY(cudaGetLastError());
    }
    if (w_running != nullptr) SLIM_CUDA_TRY(cudaMemcpyAsync(w_running, w, total * sizeof(double), cudaMemcpyDeviceToDevice, s));
    return SLIM_OK;
}

}  // extern "C"
