// Producing the layer's inputs on the device: group salience (first step of SBA) and the
// asymmetric min-max quantizer of Eq. 1.  fp64 arithmetic from fp16 weights, fixed summation
// order, so the outputs are reproducible bit for bit.  Every kernel is a template over the group
// size GS (32, 64, 128, 256, 512 columns: the sizes of the paper's group-size ablation).
#include "slim_common.cuh"

#include <cstring>

namespace slim {

// Bit-widths of up to 1024 groups, two bits each (b - 1), passed by value in kernel parameters.
constexpr int kQuantMaxGroups = 1024;
struct GroupBits {
    int G;
    uint32_t w[kQuantMaxGroups / 16];
    __host__ __device__ int at(int j) const { return 1 + static_cast<int>((w[j >> 4] >> (2 * (j & 15))) & 3u); }
};

// Validates the shape as the other entry points do and fills the table (bits_host has K / g entries).
static int make_group_bits(int N, int K, int g, const uint8_t* bits_host, GroupBits* out) {
    if (bits_host == nullptr || N < 0 || K < 0) return SLIM_ERR_INVALID_ARG;
    if (g != 32 && g != 64 && g != 128 && g != 256 && g != 512) return SLIM_ERR_UNSUPPORTED;
    // the quantizers work group by group: any K that is a multiple of g (Algorithm 1 hands them one group at a time)
    if (K % g != 0 || N % 16 != 0 || K / g > kQuantMaxGroups) return SLIM_ERR_UNSUPPORTED;
    memset(out, 0, sizeof *out);
    out->G = K / g;
    for (int j = 0; j < out->G; ++j) {
        const int b = bits_host[j];
        if (b < 1 || b > 4) return SLIM_ERR_INVALID_ARG;
        out->w[j >> 4] |= static_cast<uint32_t>(b - 1) << (2 * (j & 15));
    }
    return SLIM_OK;
}

// The CPL = GS / 32 consecutive weights of a lane, and its codes (one byte each).
template <int CPL>
__device__ __forceinline__ void load_weights(const __half* src, float (&w)[CPL]) {
    if constexpr (CPL == 1) {
        w[0] = __half2float(*src);
    } else if constexpr (CPL == 2) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(src));
        w[0] = f.x; w[1] = f.y;
    } else if constexpr (CPL == 4) {
        const uint2 raw = *reinterpret_cast<const uint2*>(src);
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        w[0] = a.x; w[1] = a.y; w[2] = b.x; w[3] = b.y;
    } else {
#pragma unroll
        for (int q = 0; q < CPL / 8; ++q) {
            const uint4 raw = reinterpret_cast<const uint4*>(src)[q];
            const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
                w[8 * q + 2 * i] = v.x; w[8 * q + 2 * i + 1] = v.y;
            }
        }
    }
}
template <int CPL>
__device__ __forceinline__ void store_codes(uint8_t* dst, const uint8_t (&q)[CPL]) {
    if constexpr (CPL == 1) {
        dst[0] = q[0];
    } else if constexpr (CPL == 2) {
        *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(q[0] | (q[1] << 8));
    } else {
#pragma unroll
        for (int v = 0; v < CPL / 4; ++v)
            reinterpret_cast<uint32_t*>(dst)[v] = q[4 * v] | (q[4 * v + 1] << 8) | (q[4 * v + 2] << 16) | (static_cast<uint32_t>(q[4 * v + 3]) << 24);
    }
}

// One cluster of kSalCluster blocks per group; block r of the cluster owns the r-th slice of the
// rows.  Thread (ph, cp) owns column pair cp (2 columns) and rows ph, ph + P, ... of the slice
// (P = 512 / GS phases, so that the 256 threads cover the GS / 2 column pairs P times).
// Column sums of squares are accumulated in fp64 in ascending row order per phase, the
// phases are added in order, the blocks' sums are added in rank order by block 0 (which receives
// them through distributed shared memory), then the GS columns are weighted by a_k^2 and summed
// in order: a fixed order, so the result is reproducible.
constexpr int kSalCluster = 8;

template <int GS>
__global__ void __cluster_dims__(kSalCluster, 1, 1) __launch_bounds__(256)
salience_kernel(const __half* __restrict__ W, const float* __restrict__ act_norm, double* __restrict__ salience, int N, int K) {
    constexpr int PAIRS = GS / 2, P = 256 / PAIRS;
    const int j = blockIdx.x / kSalCluster, r = blockIdx.x % kSalCluster;     // group, rank in the cluster
    const int cp = threadIdx.x % PAIRS, ph = threadIdx.x / PAIRS;
    const int rows = (N + kSalCluster - 1) / kSalCluster;
    const int n0 = r * rows, n1 = min(N, n0 + rows);
    const __half2* base = reinterpret_cast<const __half2*>(W + static_cast<size_t>(GS) * j) + cp;
    double s0 = 0.0, s1 = 0.0;
    for (int n = n0 + ph; n < n1; n += P) {
        const float2 v = __half22float2(base[static_cast<size_t>(n) * (K / 2)]);
        s0 += static_cast<double>(v.x) * static_cast<double>(v.x);
        s1 += static_cast<double>(v.y) * static_cast<double>(v.y);
    }
    __shared__ double part[P][GS];
    __shared__ double from_rank[kSalCluster][GS];        // used in block 0 of the cluster
    part[ph][2 * cp] = s0;
    part[ph][2 * cp + 1] = s1;
    __syncthreads();
    for (int k = threadIdx.x; k < GS; k += 256) {
        double col = part[0][k];
#pragma unroll
        for (int q = 1; q < P; ++q) col += part[q][k];
        // hand the slice's column sum to block 0
        uint32_t remote;
        const uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(&from_rank[r][k]));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0));
        asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(remote), "d"(col) : "memory");
    }
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (r == 0 && threadIdx.x == 0) {
        double total = 0.0;
        for (int k = 0; k < GS; ++k) {
            double col = 0.0;
            for (int q = 0; q < kSalCluster; ++q) col += from_rank[q][k];
            const double a = static_cast<double>(act_norm[GS * j + k]);
            total += a * a * col;
        }
        salience[j] = total;
    }
}

__device__ __forceinline__ unsigned short double_to_half_bits_rn(double v) {
    unsigned short h;
    asm("cvt.rn.f16.f64 %0, %1;" : "=h"(h) : "d"(v));
    return h;
}

// Groups a launch of the quantizer is restricted to (n = 0: all groups).
struct GroupSubset {
    int n;
    uint16_t idx[kQuantMaxGroups];
};

// rint(w / s) for fp16-exact w and s > 0 without a division per weight: t = w * (1/s) is within a few
// ulps of the quotient, and the quotient of two fp16 numbers that is not exactly half-way between
// two integers stays farther than 2^-13 from it (its denominator has at most 11 bits; |w/s| < 2^6
// here), so rint(t) is rint(w/s) unless t sits within 1e-6 of a half-integer, which can only be an
// exact tie and goes to the even neighbour as rint does.
__device__ __forceinline__ double rint_quotient(double w, double inv_s) {
    const double t = w * inv_s;
    const double k = rint(t);
    if (fabs(fabs(t - k) - 0.5) < 1e-6) {
        const double m = rint(t - 0.5);                   // the integer below the tie
        return fmod(m, 2.0) == 0.0 ? m : m + 1.0;
    }
    return k;
}

// One warp per (row, group): lane l owns the GS / 32 consecutive columns from (GS / 32) l on.  With sign_alpha != 0 the
// one-bit groups are binarised as in Eq. 2 (q = [w >= 0], alpha = mean |w|, stored as s = 2 alpha,
// z = 1/2 so that s (q - z) = +-alpha); all other groups, and all groups otherwise, use Eq. 1.
template <int GS>
__global__ void __launch_bounds__(256) quantize_minmax_kernel(const __half* __restrict__ W, uint8_t* __restrict__ codes,
                                                              __half* __restrict__ scales, __half* __restrict__ zeros,
                                                              int N, int K, int sign_alpha, GroupSubset sub, GroupBits gb) {
    constexpr int CPL = GS / 32;
    const long long warp = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int G = sub.n > 0 ? sub.n : gb.G;              // groups this launch quantises
    if (warp >= static_cast<long long>(N) * G) return;
    const int n = static_cast<int>(warp / G);
    const int j = sub.n > 0 ? sub.idx[warp % G] : static_cast<int>(warp % G);
    const size_t off = static_cast<size_t>(n) * K + GS * j + CPL * lane;
    float w[CPL];
    load_weights<CPL>(W + off, w);
    float lo = w[0], hi = w[0];
#pragma unroll
    for (int i = 1; i < CPL; ++i) { lo = fminf(lo, w[i]); hi = fmaxf(hi, w[i]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    lo = fminf(lo, 0.0f);
    hi = fmaxf(hi, 0.0f);
    const int b = gb.at(j);
    uint8_t q8[CPL];
    if (sign_alpha != 0 && b == 1) {
        // the sum of at most 512 fp16 magnitudes is exact in fp64, whatever the order
        double sum = 0.0;
#pragma unroll
        for (int i = 0; i < CPL; ++i) sum += fabs(static_cast<double>(w[i]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
#pragma unroll
        for (int i = 0; i < CPL; ++i) q8[i] = w[i] >= 0.0f ? 1 : 0;
        store_codes<CPL>(codes + off, q8);
        if (lane == 0) {
            scales[static_cast<size_t>(j) * N + n] = __ushort_as_half(double_to_half_bits_rn(sum / static_cast<double>(GS / 2)));   // 2 * mean
            zeros[static_cast<size_t>(j) * N + n] = __float2half_rn(0.5f);
        }
        return;
    }
    const double levels = static_cast<double>((1 << b) - 1);
    unsigned short sbits = double_to_half_bits_rn((static_cast<double>(hi) - static_cast<double>(lo)) / levels);
    if ((sbits & 0x7fffu) == 0x7c00u) sbits = 0x7bffu;  // beyond fp16 range -> 65504
    if ((sbits & 0x7fffu) == 0u) sbits = 0x3c00u;       // zero scale -> 1
    const __half s16 = __ushort_as_half(sbits);
    const double s = static_cast<double>(__half2float(s16));
    const double z = fmin(fmax(-rint(static_cast<double>(lo) / s), 0.0), levels);
    const double inv_s = 1.0 / s;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const double q = fmin(fmax(rint_quotient(static_cast<double>(w[i]), inv_s) + z, 0.0), levels);
        q8[i] = static_cast<uint8_t>(static_cast<int>(q));
    }
    store_codes<CPL>(codes + off, q8);
    if (lane == 0) {
        scales[static_cast<size_t>(j) * N + n] = s16;
        zeros[static_cast<size_t>(j) * N + n] = __float2half_rn(static_cast<float>(z));
    }
}

// Calls f(tag) with tag::value = g for the five group sizes.
template <int V> struct GroupSizeTag { static constexpr int value = V; };
template <typename F>
static void for_group_size(int g, F&& f) {
    switch (g) {
        case 32: f(GroupSizeTag<32>{}); break;
        case 64: f(GroupSizeTag<64>{}); break;
        case 128: f(GroupSizeTag<128>{}); break;
        case 256: f(GroupSizeTag<256>{}); break;
        default: f(GroupSizeTag<512>{}); break;
    }
}

}  // namespace slim

extern "C" {

int slim_group_salience(const void* W, const float* act_norm, double* salience, int N, int K, int g, void* stream) {
    if (N < 0 || K < 0) return SLIM_ERR_INVALID_ARG;
    if (g != 32 && g != 64 && g != 128 && g != 256 && g != 512) return SLIM_ERR_UNSUPPORTED;
    if (K % g != 0 || K / g > slim::kQuantMaxGroups) return SLIM_ERR_UNSUPPORTED;
    if (K == 0) return SLIM_OK;
    if (W == nullptr || act_norm == nullptr || salience == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(W) || !slim::aligned16(act_norm) || !slim::aligned16(salience)) return SLIM_ERR_ALIGNMENT;
    slim::for_group_size(g, [&](auto tag) {
        slim::salience_kernel<decltype(tag)::value><<<slim::kSalCluster * (K / g), 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __half*>(W), act_norm, salience, N, K);
    });
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

static int quantize_minmax_impl(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                                int N, int K, int g, int sign_alpha, const int* groups_host, int n_groups, void* stream) {
    slim::GroupBits gb;
    const int st = slim::make_group_bits(N, K, g, bits_host, &gb);
    if (st != SLIM_OK) return st;
    if (N == 0 || K == 0) return SLIM_OK;
    if (W == nullptr || codes == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(W) || !slim::aligned16(codes) || !slim::aligned16(scales) || !slim::aligned16(zeros))
        return SLIM_ERR_ALIGNMENT;
    slim::GroupSubset sub;
    memset(&sub, 0, sizeof sub);
    if (groups_host != nullptr) {
        if (n_groups < 0 || n_groups > gb.G) return SLIM_ERR_INVALID_ARG;
        if (n_groups == 0) return SLIM_OK;
        for (int i = 0; i < n_groups; ++i) {
            if (groups_host[i] < 0 || groups_host[i] >= gb.G) return SLIM_ERR_INVALID_ARG;
            sub.idx[i] = static_cast<uint16_t>(groups_host[i]);
        }
        sub.n = n_groups;
    }
    const long long warps = static_cast<long long>(N) * (sub.n > 0 ? sub.n : gb.G);
    const unsigned grid = static_cast<unsigned>((warps + 7) / 8);
    slim::for_group_size(g, [&](auto tag) {
        slim::quantize_minmax_kernel<decltype(tag)::value><<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __half*>(W), codes, static_cast<__half*>(scales), static_cast<__half*>(zeros), N, K, sign_alpha, sub, gb);
    });
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}


int slim_quantize_minmax(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                         int N, int K, int g, void* stream) {
    return quantize_minmax_impl(W, bits_host, codes, scales, zeros, N, K, g, 0, nullptr, 0, stream);
}

int slim_quantize_minmax_groups(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                                int N, int K, int g, const int* groups_host, int n_groups, void* stream) {
    if (groups_host == nullptr) return SLIM_ERR_INVALID_ARG;
    return quantize_minmax_impl(W, bits_host, codes, scales, zeros, N, K, g, 0, groups_host, n_groups, stream);
}

int slim_quantize_minmax_sign1(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                               int N, int K, int g, void* stream) {
    return quantize_minmax_impl(W, bits_host, codes, scales, zeros, N, K, g, 1, nullptr, 0, stream);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------ SQC
// Salience-Weighted Quantizer Calibration (Sec. 3.3, Eq. 5; function SQC of Algorithm 2).
// One warp per (row, group): the group's weights sit in shared memory as fp64, every lane evaluates
// the candidates tau_i with i = lane, lane + 32, ... one after another, walking the columns in
// order, so that every loss is the same fp64 sum a sequential program would form.  Every fp64
// operation is an explicit round-to-nearest intrinsic: nothing may be contracted into an FMA.
namespace slim {

constexpr int kSqcWarps = 4;

struct SqcBest {
    double loss;
    int idx;
};

template <int GS>
__global__ void __launch_bounds__(kSqcWarps * 32) quantize_sqc_kernel(const __half* __restrict__ W, uint8_t* __restrict__ codes,
                                                                       __half* __restrict__ scales, __half* __restrict__ zeros,
                                                                       int* __restrict__ tau_index, int N, int K, double lambda,
                                                                       int n_half, GroupBits gb) {
    constexpr int CPL = GS / 32;
    __shared__ double sw[kSqcWarps][GS];
    const int lane = threadIdx.x & 31, wl = threadIdx.x >> 5;
    const long long pair = static_cast<long long>(blockIdx.x) * kSqcWarps + wl;
    const int G = gb.G;
    if (pair >= static_cast<long long>(N) * G) return;
    const int n = static_cast<int>(pair / G), j = static_cast<int>(pair % G);
    const size_t off = static_cast<size_t>(n) * K + GS * j + CPL * lane;
    float w4[CPL];
    load_weights<CPL>(W + off, w4);
    float lo = w4[0], hi = w4[0];
#pragma unroll
    for (int i = 1; i < CPL; ++i) { lo = fminf(lo, w4[i]); hi = fmaxf(hi, w4[i]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    const double dlo = static_cast<double>(fminf(lo, 0.0f)), dhi = static_cast<double>(fmaxf(hi, 0.0f));
#pragma unroll
    for (int i = 0; i < CPL; ++i) sw[wl][CPL * lane + i] = static_cast<double>(w4[i]);
    __syncwarp();
    const double* w = sw[wl];

    // 3-sigma mask: mean and population standard deviation, both sums in column order
    double tot = 0.0;
#pragma unroll 4
    for (int k = 0; k < GS; ++k) tot = __dadd_rn(tot, w[k]);
    const double mu = __ddiv_rn(tot, static_cast<double>(GS));
    double var = 0.0;
#pragma unroll 4
    for (int k = 0; k < GS; ++k) {
        const double d = __dsub_rn(w[k], mu);
        var = __dadd_rn(var, __dmul_rn(d, d));
    }
    const double sd = __dsqrt_rn(__ddiv_rn(var, static_cast<double>(GS)));
    const double t_lo = __dsub_rn(mu, __dmul_rn(3.0, sd)), t_hi = __dadd_rn(mu, __dmul_rn(3.0, sd));

    const int b = gb.at(j);
    const double levels = static_cast<double>((1 << b) - 1);
    const double tau0 = __dsub_rn(1.0, lambda), step = __ddiv_rn(lambda, static_cast<double>(n_half));
    const double range = __dsub_rn(dhi, dlo);

    // scale (fp16 bits) and zero point of candidate i
    auto candidate = [&](int i, double* s_out, double* z_out) -> unsigned short {
        const double tau = __dadd_rn(tau0, __dmul_rn(static_cast<double>(i), step));
        unsigned short sbits = double_to_half_bits_rn(__ddiv_rn(__dmul_rn(tau, range), levels));
        if ((sbits & 0x7fffu) == 0x7c00u) sbits = 0x7bffu;  // beyond fp16 range -> 65504
        if ((sbits & 0x7fffu) == 0u) sbits = 0x3c00u;       // zero scale -> 1
        const double s = static_cast<double>(__half2float(__ushort_as_half(sbits)));
        *s_out = s;
        *z_out = fmin(fmax(-rint(__ddiv_rn(__dmul_rn(tau, dlo), s)), 0.0), levels) + 0.0;
        return sbits;
    };

    SqcBest best{__longlong_as_double(0x7ff0000000000000ll), 0x7fffffff};
    for (int i = lane; i < 2 * n_half; i += 32) {
        double s, z;
        (void)candidate(i, &s, &z);
        const double inv_s = __ddiv_rn(1.0, s);           // |w / s| < 2^6 here too: see rint_quotient
        double Ls = 0.0, Lus = 0.0;
#pragma unroll 2
        for (int k = 0; k < GS; ++k) {
            const double wk = w[k];
            const double q = fmin(fmax(__dadd_rn(rint_quotient(wk, inv_s), z), 0.0), levels);
            const double e = __dsub_rn(wk, __dmul_rn(s, __dsub_rn(q, z)));
            const double sq = __dmul_rn(e, e);
            if (wk < t_lo || wk > t_hi) Ls = __dadd_rn(Ls, sq);
            else Lus = __dadd_rn(Lus, sq);
        }
        const double total = __dadd_rn(Ls, Lus);
        if (total < best.loss) { best.loss = total; best.idx = i; }   // strict: the first candidate wins ties
    }
    // smallest loss over the warp, smallest index among equals
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ol = __shfl_xor_sync(0xffffffffu, best.loss, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best.idx, o);
        if (ol < best.loss || (ol == best.loss && oi < best.idx)) { best.loss = ol; best.idx = oi; }
    }
    double s, z;
    const unsigned short sbits = candidate(best.idx, &s, &z);
    uint8_t q8[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const double q = fmin(fmax(__dadd_rn(rint(__ddiv_rn(static_cast<double>(w4[i]), s)), z), 0.0), levels);
        q8[i] = static_cast<uint8_t>(static_cast<int>(q));
    }
    store_codes<CPL>(codes + off, q8);
    if (lane == 0) {
        scales[static_cast<size_t>(j) * N + n] = __ushort_as_half(sbits);
        zeros[static_cast<size_t>(j) * N + n] = __float2half_rn(static_cast<float>(z));
        if (tau_index != nullptr) tau_index[static_cast<size_t>(j) * N + n] = best.idx;
    }
}

}  // namespace slim

extern "C" int slim_quantize_sqc(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                                 int* tau_index, int N, int K, int g, double lambda, int n, void* stream) {
    slim::GroupBits gb;
    const int st = slim::make_group_bits(N, K, g, bits_host, &gb);
    if (st != SLIM_OK) return st;
    if (!(lambda >= 0.0 && lambda < 1.0) || n < 1 || n > 64) return SLIM_ERR_INVALID_ARG;
    if (N == 0 || K == 0) return SLIM_OK;
    if (W == nullptr || codes == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(W) || !slim::aligned16(codes) || !slim::aligned16(scales) || !slim::aligned16(zeros) ||
        (tau_index != nullptr && !slim::aligned16(tau_index)))
        return SLIM_ERR_ALIGNMENT;
    const long long pairs = static_cast<long long>(N) * gb.G;
    const unsigned grid = static_cast<unsigned>((pairs + slim::kSqcWarps - 1) / slim::kSqcWarps);
    slim::for_group_size(g, [&](auto tag) {
        slim::quantize_sqc_kernel<decltype(tag)::value><<<grid, slim::kSqcWarps * 32, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __half*>(W), codes, static_cast<__half*>(scales), static_cast<__half*>(zeros), tau_index, N, K,
            lambda, n, gb);
    });
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}
