// slim_sba_search: Salience-Determined Bit Allocation, func SBA of Algorithm 2 (Sec. 3.2.2, Eq. 4).
//
// For p = 0 (uniform), 1, ..., floor(G/2) the p most salient groups get N-bar+1 bits and the p least
// salient N-bar-1; the weight is quantised with Eq. 1 under that map and the candidate's error is
// the KL divergence between softmax(x w^T) and softmax(x w-hat^T), averaged over the calibration
// tokens; the first p with the smallest error wins.  Every step runs in this library's kernels:
//   salience            slim_group_salience            (first step of func SBA)
//   x w^T               dense_linear_kernel            (fp16 in, fp32 accumulate on mma.sync, fp32 out; once)
//   quantise, pack      slim_quantize_minmax (first candidate), slim_quantize_minmax_groups (the two groups
//                       that change from one candidate to the next), slim_pack_weights
//   x w-hat^T           slim_mpq_gemv / slim_mpq_gemm  (the hot path itself evaluates the candidate)
//   error               softmax_kl_kernel              (fp64, fixed reduction order)
// The host only ranks the G saliences, loops over p and takes the minimum of G/2 + 1 numbers.
#include "slim_common.cuh"

#include <cstring>

namespace slim {

// ------------------------------------------------------------------------------------------ x w^T, full precision
// y[m][n] = sum_k x[m][k] * W[n][k]: fp16 operands, fp32 accumulation on the tensor cores
// (mma.sync m16n8k16; it runs once per layer).  A block of four warps takes 64 tokens x 64 rows, warp w
// the tokens 16w .. 16w+15; operand fragments are read straight from global memory (x and W are
// both k-contiguous, which is what the row x column fragment layouts want).
constexpr int kDenseTile = 64;
constexpr int kDenseK = 32;      // K must be a multiple of this

__global__ void __launch_bounds__(128) dense_linear_kernel(const __half* __restrict__ x, const __half* __restrict__ W,
                                                           float* __restrict__ y, int M, int N, int K) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, c = lane & 3;
    const int m0 = blockIdx.y * kDenseTile + 16 * warp, n0 = blockIdx.x * kDenseTile;
    // rows past the ends are clamped for the loads and masked at the store
    const int ma = min(m0 + gq, M - 1), mb = min(m0 + gq + 8, M - 1);
    const uint32_t* xa = reinterpret_cast<const uint32_t*>(x + static_cast<size_t>(ma) * K) + c;
    const uint32_t* xb = reinterpret_cast<const uint32_t*>(x + static_cast<size_t>(mb) * K) + c;
    const uint32_t* wr[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) wr[t] = reinterpret_cast<const uint32_t*>(W + static_cast<size_t>(min(n0 + 8 * t + gq, N - 1)) * K) + c;
    float acc[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[t][r] = 0.f;
    for (int k0 = 0; k0 < K; k0 += 16) {
        const int o = k0 >> 1;                             // in 32-bit words
        const uint32_t a0 = __ldg(xa + o), a1 = __ldg(xb + o), a2 = __ldg(xa + o + 4), a3 = __ldg(xb + o + 4);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t b0 = __ldg(wr[t] + o), b1 = __ldg(wr[t] + o + 4);
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+f"(acc[t][0]), "+f"(acc[t][1]), "+f"(acc[t][2]), "+f"(acc[t][3])
                         : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
    // D fragment: rows (tokens) gq and gq + 8, columns (weight rows) 2c and 2c + 1 of each 8-wide tile
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int n = n0 + 8 * t + 2 * c;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int m = m0 + gq + 8 * h;
            if (m < M) {
                if (n < N) y[static_cast<size_t>(m) * N + n] = acc[t][2 * h];
                if (n + 1 < N) y[static_cast<size_t>(m) * N + n + 1] = acc[t][2 * h + 1];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ softmax + KL
// Block tree reduction in a fixed order (deterministic); every thread gets the result.
template <typename T, typename Op>
__device__ __forceinline__ T block_reduce(T v, T* scratch, Op op) {
    const int tid = threadIdx.x;
    scratch[tid] = v;
    __syncthreads();
    for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
        if (tid < s) scratch[tid] = op(scratch[tid], scratch[tid + s]);
        __syncthreads();
    }
    const T r = scratch[0];
    __syncthreads();
    return r;
}

// One block per token: kl[t] = sum_n p_n (log p_n - log q_n), p = softmax(y_ref[t]), q = softmax(y_q[t]).
__global__ void __launch_bounds__(256) softmax_kl_kernel(const float* __restrict__ y_ref, const __half* __restrict__ y_q,
                                                         double* __restrict__ kl, int N) {
    __shared__ double scratch[256];
    const int t = blockIdx.x, tid = threadIdx.x;
    const float* a = y_ref + static_cast<size_t>(t) * N;
    const __half* b = y_q + static_cast<size_t>(t) * N;
    double ma = -1.0e300, mb = -1.0e300;
    for (int n = tid; n < N; n += 256) {
        ma = fmax(ma, static_cast<double>(a[n]));
        mb = fmax(mb, static_cast<double>(__half2float(b[n])));
    }
    auto mx = [](double u, double v) { return fmax(u, v); };
    auto add = [](double u, double v) { return u + v; };
    ma = block_reduce(ma, scratch, mx);
    mb = block_reduce(mb, scratch, mx);
    double sa = 0.0, sb = 0.0;
    for (int n = tid; n < N; n += 256) {
        sa += exp(static_cast<double>(a[n]) - ma);
        sb += exp(static_cast<double>(__half2float(b[n])) - mb);
    }
    sa = block_reduce(sa, scratch, add);
    sb = block_reduce(sb, scratch, add);
    const double la = ma + log(sa), lb = mb + log(sb);       // log of the two partition sums
    double d = 0.0;
    for (int n = tid; n < N; n += 256) {
        const double lp = static_cast<double>(a[n]) - la, lq = static_cast<double>(__half2float(b[n])) - lb;
        d += exp(lp) * (lp - lq);
    }
    d = block_reduce(d, scratch, add);
    if (tid == 0) kl[t] = d;
}

// ------------------------------------------------------------------------------------------ workspace layout
struct SbaLayout {
    size_t linear_ws, linear_ws_bytes;   // workspace of slim_mpq_gemv / slim_mpq_gemm (status word first)
    size_t salience, codes, scales, zeros, packed, y_ref, y_q, kl;
    size_t total;
    int candidates;
};
static size_t up256(size_t v) { return (v + 255) / 256 * 256; }

constexpr int kSbaMaxGroups = 1024;       // K <= 32768 in groups of 32 columns

static int sba_layout(int M, int N, int K, int g, int avg_bits, SbaLayout* lay) {
    if (M < 1 || N < 16 || K < SLIM_GROUP || avg_bits < 2 || avg_bits > 3) return SLIM_ERR_INVALID_ARG;
    if (g != 32 && g != 64 && g != 128 && g != 256 && g != 512) return SLIM_ERR_UNSUPPORTED;
    if (K % g != 0 || K % SLIM_GROUP != 0 || N % 16 != 0 || K / SLIM_GROUP > SLIM_MAX_GROUPS) return SLIM_ERR_UNSUPPORTED;
    const int G = K / g;
    uint8_t widest[kSbaMaxGroups];
    for (int j = 0; j < G; ++j) widest[j] = 3;      // 3-bit groups have two slices: the largest staging area of any map
    size_t need = 0;
    const int st = slim_workspace_bytes(M, N, K, g, widest, &need);     // every candidate map needs at most this
    if (st != SLIM_OK) return st;
    size_t o = 0;
    lay->linear_ws = o;  lay->linear_ws_bytes = up256(need);  o += lay->linear_ws_bytes;
    lay->salience = o;   o += up256(static_cast<size_t>(G) * sizeof(double));
    lay->codes = o;      o += up256(static_cast<size_t>(N) * K);
    lay->scales = o;     o += up256(static_cast<size_t>(G) * N * 2);
    lay->zeros = o;      o += up256(static_cast<size_t>(G) * N * 2);
    lay->packed = o;     o += up256(static_cast<size_t>(N) * K / 8 * (avg_bits + 1));
    lay->y_ref = o;      o += up256(static_cast<size_t>(M) * N * sizeof(float));
    lay->y_q = o;        o += up256(static_cast<size_t>(M) * N * 2);
    lay->candidates = G / 2 + 1;
    lay->kl = o;         o += up256(static_cast<size_t>(lay->candidates) * M * sizeof(double));
    lay->total = o;
    return SLIM_OK;
}

}  // namespace slim

extern "C" {

int slim_sba_workspace_bytes(int M, int N, int K, int g, int avg_bits, size_t* out_bytes) {
    if (out_bytes == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::SbaLayout lay;
    const int st = slim::sba_layout(M, N, K, g, avg_bits, &lay);
    if (st != SLIM_OK) return st;
    *out_bytes = lay.total;
    return SLIM_OK;
}

int slim_dense_linear(const void* x, const void* W, float* y, int M, int N, int K, void* stream) {
    if (M < 0 || N < 0 || K < 0 || K % 8 != 0) return SLIM_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SLIM_OK;
    if (x == nullptr || W == nullptr || y == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(x) || !slim::aligned16(W) || !slim::aligned16(y)) return SLIM_ERR_ALIGNMENT;
    if (K % slim::kDenseK != 0) return SLIM_ERR_UNSUPPORTED;
    const dim3 grid((N + slim::kDenseTile - 1) / slim::kDenseTile, (M + slim::kDenseTile - 1) / slim::kDenseTile);
    slim::dense_linear_kernel<<<grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(x), static_cast<const __half*>(W), y, M, N, K);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int slim_softmax_kl(const float* y_ref, const void* y_q, double* kl, int M, int N, void* stream) {
    if (M < 0 || N < 1) return SLIM_ERR_INVALID_ARG;
    if (M == 0) return SLIM_OK;
    if (y_ref == nullptr || y_q == nullptr || kl == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::softmax_kl_kernel<<<M, 256, 0, static_cast<cudaStream_t>(stream)>>>(y_ref, static_cast<const __half*>(y_q), kl, N);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int slim_sba_search(const void* W, const void* x, const float* act_norm, int M, int N, int K, int g, int avg_bits,
                    int include_uniform, void* workspace, size_t workspace_bytes,
                    int* p_star_host, uint8_t* bits_host_out, double* errors_host, void* stream) {
    if (p_star_host == nullptr || bits_host_out == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::SbaLayout lay;
    int st = slim::sba_layout(M, N, K, g, avg_bits, &lay);
    if (st != SLIM_OK) return st;
    if (W == nullptr || x == nullptr || act_norm == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(W) || !slim::aligned16(x)) return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < lay.total) return SLIM_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SLIM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int G = K / g;
    const int first = include_uniform ? 0 : 1;
    if (first > G / 2) return SLIM_ERR_INVALID_ARG;                       // a single group has only the uniform map

    // salience and its ranking (host: G numbers)
    double sal[slim::kSbaMaxGroups];
    double* sal_dev = reinterpret_cast<double*>(ws + lay.salience);
    st = slim_group_salience(W, act_norm, sal_dev, N, K, g, stream);
    if (st != SLIM_OK) return st;
    SLIM_CUDA_TRY(cudaMemcpyAsync(sal, sal_dev, static_cast<size_t>(G) * sizeof(double), cudaMemcpyDeviceToHost, s));
    SLIM_CUDA_TRY(cudaStreamSynchronize(s));

    // reference output, once
    float* y_ref = reinterpret_cast<float*>(ws + lay.y_ref);
    st = slim_dense_linear(x, W, y_ref, M, N, K, stream);
    if (st != SLIM_OK) return st;
    st = slim_workspace_init(ws + lay.linear_ws, lay.linear_ws_bytes, stream);
    if (st != SLIM_OK) return st;

    uint8_t* codes = ws + lay.codes;
    void* scales = ws + lay.scales;
    void* zeros = ws + lay.zeros;
    void* packed = ws + lay.packed;
    void* y_q = ws + lay.y_q;
    double* kl = reinterpret_cast<double*>(ws + lay.kl);
    uint8_t bits[slim::kSbaMaxGroups], prev[slim::kSbaMaxGroups];
    for (int p = first; p <= G / 2; ++p) {
        st = slim_allocate_bits(sal, G, avg_bits, p, bits);
        if (st != SLIM_OK) return st;
        if (p == first) {
            st = slim_quantize_minmax(W, bits, codes, scales, zeros, N, K, g, stream);
        } else {
            // consecutive candidates differ in the two groups the double pointer has just passed: only those
            // are quantised again, the codes, scales and zeros of all other groups stay
            int changed[slim::kSbaMaxGroups], n_changed = 0;
            for (int j = 0; j < G; ++j)
                if (bits[j] != prev[j]) changed[n_changed++] = j;
            st = slim_quantize_minmax_groups(W, bits, codes, scales, zeros, N, K, g, changed, n_changed, stream);
        }
        if (st != SLIM_OK) return st;
        memcpy(prev, bits, sizeof prev);
        st = slim_pack_weights(codes, bits, packed, N, K, g, stream);
        if (st != SLIM_OK) return st;
        st = M <= SLIM_GEMV_MAX_M
                 ? slim_mpq_gemv(x, packed, bits, scales, zeros, y_q, M, N, K, g, ws + lay.linear_ws, lay.linear_ws_bytes, stream)
                 : slim_mpq_gemm(x, packed, bits, scales, zeros, y_q, M, N, K, g, ws + lay.linear_ws, lay.linear_ws_bytes, stream);
        if (st != SLIM_OK) return st;
        st = slim_softmax_kl(y_ref, y_q, kl + static_cast<size_t>(p - first) * M, M, N, stream);
        if (st != SLIM_OK) return st;
    }
    st = slim_workspace_status(ws + lay.linear_ws, stream);               // synchronises; a device-side time-out shows here
    if (st != SLIM_OK) return st;

    // mean over the tokens in token order, first minimum over p
    const int P = G / 2 + 1 - first;
    int best = 0;
    double best_err = 0.0;
    for (int i = 0; i < P; ++i) {
        double host_kl[256];
        double sum = 0.0;
        for (int m0 = 0; m0 < M; m0 += 256) {
            const int n = M - m0 < 256 ? M - m0 : 256;
            SLIM_CUDA_TRY(cudaMemcpy(host_kl, kl + static_cast<size_t>(i) * M + m0, static_cast<size_t>(n) * sizeof(double),
                                     cudaMemcpyDeviceToHost));
            for (int m = 0; m < n; ++m) sum += host_kl[m];
        }
        const double err = sum / M;
        if (errors_host != nullptr) errors_host[i] = err;
        if (i == 0 || err < best_err) { best = i; best_err = err; }
    }
    *p_star_host = first + best;
    return slim_allocate_bits(sal, G, avg_bits, first + best, bits_host_out);
}

}  // extern "C"
