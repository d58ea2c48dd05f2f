// Group sizes of 32 and 64 columns (the small end of the paper's group-size ablation, appendix).
//
// The K-tile of the packed format is the group itself (T = g columns): a tile of b bits takes N*T*b/8 bytes and holds,
// per 16-row tile, b units of 2T bytes; a unit is 32 lanes x T/16 bytes, lane 4*gq + c holding one item of T/4 bits
// for each of the rows 2gq and 2gq + 1 (the column range c of the group); an item of a width-w slice has (T/4)/w
// fields.  This is the 128-column layout with every 32 replaced by T/4, so the decode below is the same bit
// shuffling on 8- and 16-bit items.
//
// These group sizes trade a fifth to a half more scale and zero-point bytes for accuracy; they are served by plain
// CUDA-core kernels (one FMA per weight and token), not by the tensor-core kernels of the 128-column tiles:
//   pack_small_kernel, dequant_small_kernel   one thread per item / per 8 outputs, bit-exact
//   gemv_small_kernel (1 <= M <= 16)          a block per 16-row tile, the groups dealt to its 16 warps, fp32 accumulation
//   M > 16                                    the weights are materialised as fp16 in the workspace (dequant_small_kernel)
//                                             and multiplied by dense_f16_kernel (mma.sync, fp32 accumulation)
#include "slim_common.cuh"

#include <cstring>

namespace slim {

constexpr int kSmallMaxGroups = 1024;

struct SmallTable {
    int G, T;                                   // groups, columns per group
    uint16_t prefix[kSmallMaxGroups + 1];       // bits of the groups before j
    uint8_t bits[kSmallMaxGroups];
};

static int make_small_table(int N, int K, int g, const uint8_t* bits_host, SmallTable* out) {
    if (bits_host == nullptr || N < 0 || K < 0) return SLIM_ERR_INVALID_ARG;
    if (!is_small_group(g) || K % SLIM_GROUP != 0 || N % 16 != 0 || K / g > kSmallMaxGroups) return SLIM_ERR_UNSUPPORTED;
    out->G = K / g;
    out->T = g;
    int acc = 0;
    for (int j = 0; j < out->G; ++j) {
        const int b = bits_host[j];
        if (b < 1 || b > 4) return SLIM_ERR_INVALID_ARG;
        out->bits[j] = static_cast<uint8_t>(b);
        out->prefix[j] = static_cast<uint16_t>(acc);
        acc += b;
    }
    out->prefix[out->G] = static_cast<uint16_t>(acc);
    return SLIM_OK;
}

// Byte offset of an item: group j, 16-row tile t, unit, lane, row parity.
template <int T>
__device__ __forceinline__ size_t small_item_offset(int N, const SmallTable& st, int j, int t, int unit, int lane, int half) {
    return static_cast<size_t>(T / 8) * N * st.prefix[j] + static_cast<size_t>(t) * 2 * T * st.bits[j] + 2 * T * unit + (T / 16) * lane +
           (T / 32) * half;
}
template <int T> struct SmallItem;
template <> struct SmallItem<32> { typedef uint8_t type; };
template <> struct SmallItem<64> { typedef uint16_t type; };

// ------------------------------------------------------------------------------------------ pack
// One thread per item.  grid.y = group, grid.x covers the 4*N*b items of the widest group.
template <int T>
__global__ void __launch_bounds__(256) pack_small_kernel(const uint8_t* __restrict__ codes, uint8_t* __restrict__ packed, int N, int K,
                                                         const __grid_constant__ SmallTable st) {
    typedef typename SmallItem<T>::type item_t;
    const int j = blockIdx.y;
    const int b = st.bits[j];
    const long long ii = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;      // item inside the group
    if (ii >= 4ll * N * b) return;
    const int per_tile = 64 * b;
    const int t = static_cast<int>(ii / per_tile), rem = static_cast<int>(ii % per_tile);
    const int unit = rem >> 6, lane = (rem & 63) >> 1, half = rem & 1;
    const int s = (b == 3 && unit >= 2) ? 1 : 0;
    const int lo = slice_lo(b, s), w = slice_w(b, s), u = unit - slice_unit0(b, s);
    const int nf = T / 4 / w;
    const int c = lane & 3, gq = lane >> 2;
    const uint8_t* src = codes + static_cast<size_t>(16 * t + 2 * gq + half) * K + T * j + (T / 4) * c + nf * u;
    const uint32_t mask = (1u << w) - 1u;
    uint32_t item = 0;
    for (int f = 0; f < nf; ++f) item |= ((static_cast<uint32_t>(src[f]) >> lo) & mask) << (w * f);
    *reinterpret_cast<item_t*>(packed + small_item_offset<T>(N, st, j, t, unit, lane, half)) = static_cast<item_t>(item);
}

// Code of (row, column kk of group j) from its items.
template <int T>
__device__ __forceinline__ uint32_t small_code(const uint8_t* __restrict__ packed, int N, const SmallTable& st, int j, int row, int kk) {
    typedef typename SmallItem<T>::type item_t;
    const int b = st.bits[j];
    const int t = row >> 4, r = row & 15, gq = r >> 1, half = r & 1;
    const int c = kk / (T / 4), rem = kk % (T / 4);
    uint32_t q = 0;
    for (int s = 0; s < slice_count(b); ++s) {
        const int lo = slice_lo(b, s), w = slice_w(b, s), nf = T / 4 / w;
        const int u = rem / nf, f = rem % nf;
        const uint32_t item = *reinterpret_cast<const item_t*>(packed + small_item_offset<T>(N, st, j, t, slice_unit0(b, s) + u, 4 * gq + c, half));
        q |= ((item >> (w * f)) & ((1u << w) - 1u)) << lo;
    }
    return q;
}

// ------------------------------------------------------------------------------------------ dequant
// One thread per 8 consecutive columns of one row: W = fp16_rn(f32(s) * (f32(q) - f32(z))), as slim_dequant defines it.
template <int T>
__global__ void __launch_bounds__(256) dequant_small_kernel(const uint8_t* __restrict__ packed, const __half* __restrict__ scales,
                                                            const __half* __restrict__ zeros, __half* __restrict__ W, int N, int K,
                                                            const __grid_constant__ SmallTable st) {
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int per_row = K / 8;
    if (idx >= static_cast<long long>(N) * per_row) return;
    const int row = static_cast<int>(idx / per_row), k0 = static_cast<int>(idx % per_row) * 8;
    const int j = k0 / T, kk = k0 % T;
    const float sc = __half2float(scales[static_cast<size_t>(j) * N + row]);
    const float zp = __half2float(zeros[static_cast<size_t>(j) * N + row]);
    __align__(16) __half out[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        out[i] = __float2half_rn(__fmul_rn(sc, __fsub_rn(static_cast<float>(small_code<T>(packed, N, st, j, row, kk + i)), zp)));
    *reinterpret_cast<uint4*>(W + static_cast<size_t>(row) * K + k0) = *reinterpret_cast<const uint4*>(out);
}

// ------------------------------------------------------------------------------------------ decode path, 1 <= M <= 16
// A block of 16 warps per 16-row tile; warp w takes the groups w, w + 16, ...; lane 4*gq + c holds the items of rows
// 2gq, 2gq + 1 for the column range c of the group, decodes its T/4 codes per row and multiplies them with the
// tokens' activations (fp32 FMAs); per (row, group) acc += s * (sum_k q x - z * sum_k x).  The four lanes of a row
// pair are added by shuffles, the sixteen warps through shared memory, in a fixed order.
// The kernel is a chain of small loads, so a group's bytes (its b units, both rows of a lane in one load, and the
// scale and zero-point pairs) are requested one group ahead of their use.
constexpr int kSmallWarps = 16;

template <int T>
struct SmallRaw {
    uint32_t unit[4];      // the lane's items of rows 2gq (low part) and 2gq + 1 of up to four units
    uint32_t s2, z2;       // scales and zero points of the two rows (half2)
    int b;
};
template <int T>
__device__ __forceinline__ SmallRaw<T> small_load(const uint8_t* __restrict__ packed, const __half* __restrict__ scales,
                                                  const __half* __restrict__ zeros, int N, const SmallTable& st, int j, int t, int lane,
                                                  int row0) {
    typedef typename SmallItem<T>::type item_t;
    SmallRaw<T> r;
    r.b = st.bits[j];
    const uint8_t* base = packed + small_item_offset<T>(N, st, j, t, 0, lane, 0);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        r.unit[u] = 0u;
        if (u < r.b) {
            if (sizeof(item_t) == 1) r.unit[u] = *reinterpret_cast<const uint16_t*>(base + 2 * T * u);
            else r.unit[u] = *reinterpret_cast<const uint32_t*>(base + 2 * T * u);
        }
    }
    r.s2 = *reinterpret_cast<const uint32_t*>(scales + static_cast<size_t>(j) * N + row0);
    r.z2 = *reinterpret_cast<const uint32_t*>(zeros + static_cast<size_t>(j) * N + row0);
    return r;
}
// The codes of one lane (rows 2gq, 2gq + 1, its T/4 columns) from the W units of a width-W slice that start at unit `u0`.
template <int T, int W>
__device__ __forceinline__ void small_decode(const SmallRaw<T>& raw, int u0, int lo, uint32_t (&q)[2][T / 4]) {
    typedef typename SmallItem<T>::type item_t;
    constexpr int NF = T / 4 / W, IB = 8 * sizeof(item_t);
    constexpr uint32_t kMask = (1u << W) - 1u;
#pragma unroll
    for (int u = 0; u < W; ++u) {
        const uint32_t i0 = raw.unit[u0 + u] & ((1u << IB) - 1u), i1 = raw.unit[u0 + u] >> IB;
#pragma unroll
        for (int f = 0; f < NF; ++f) {
            q[0][NF * u + f] |= ((i0 >> (W * f)) & kMask) << lo;
            q[1][NF * u + f] |= ((i1 >> (W * f)) & kMask) << lo;
        }
    }
}

template <int T, int MT>     // MT: tokens handled per pass (the block loops over the token tiles)
__global__ void __launch_bounds__(32 * kSmallWarps, MT == 1 ? 2 : 1) gemv_small_kernel(const __half* __restrict__ x, const uint8_t* __restrict__ packed,
                                                                      const __half* __restrict__ scales, const __half* __restrict__ zeros,
                                                                      __half* __restrict__ y, int M, int N, int K,
                                                                      const __grid_constant__ SmallTable st) {
    constexpr int C = T / 4;                               // columns per lane
    __shared__ float red[kSmallWarps][MT][16];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, c = lane & 3;
    const int t = blockIdx.x;
    const int row0 = 16 * t + 2 * gq;
    for (int m0 = 0; m0 < M; m0 += MT) {
        float acc[MT][2];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m][0] = acc[m][1] = 0.f;
        SmallRaw<T> next;
        if (warp < st.G) next = small_load<T>(packed, scales, zeros, N, st, warp, t, lane, row0);
        for (int j = warp; j < st.G; j += kSmallWarps) {
            const SmallRaw<T> raw = next;
            if (j + kSmallWarps < st.G) next = small_load<T>(packed, scales, zeros, N, st, j + kSmallWarps, t, lane, row0);
            uint32_t q[2][C];
#pragma unroll
            for (int i = 0; i < C; ++i) q[0][i] = q[1][i] = 0u;
            switch (raw.b) {
                case 1: small_decode<T, 1>(raw, 0, 0, q); break;
                case 2: small_decode<T, 2>(raw, 0, 0, q); break;
                case 3: small_decode<T, 2>(raw, 0, 0, q); small_decode<T, 1>(raw, 2, 2, q); break;
                default: small_decode<T, 4>(raw, 0, 0, q); break;
            }
            const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&raw.s2));
            const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&raw.z2));
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (m0 + m >= M) break;
                const uint4* xp = reinterpret_cast<const uint4*>(x + static_cast<size_t>(m0 + m) * K + T * j + C * c);
                float d0 = 0.f, d1 = 0.f, sx = 0.f;
#pragma unroll
                for (int v = 0; v < C / 8; ++v) {
                    const uint4 xv4 = xp[v];
                    const uint32_t w4[4] = {xv4.x, xv4.y, xv4.z, xv4.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 xv = __half22float2(*reinterpret_cast<const __half2*>(&w4[i]));
                        d0 = fmaf(static_cast<float>(q[0][8 * v + 2 * i]), xv.x, d0);
                        d1 = fmaf(static_cast<float>(q[1][8 * v + 2 * i]), xv.x, d1);
                        d0 = fmaf(static_cast<float>(q[0][8 * v + 2 * i + 1]), xv.y, d0);
                        d1 = fmaf(static_cast<float>(q[1][8 * v + 2 * i + 1]), xv.y, d1);
                        sx += xv.x;
                        sx += xv.y;
                    }
                }
                acc[m][0] = fmaf(sf.x, fmaf(-zf.x, sx, d0), acc[m][0]);
                acc[m][1] = fmaf(sf.y, fmaf(-zf.y, sx, d1), acc[m][1]);
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float v = acc[m][h];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                if (c == 0) red[warp][m][2 * gq + h] = v;
            }
        }
        __syncthreads();
        for (int e = threadIdx.x; e < MT * 16; e += blockDim.x) {
            const int m = e >> 4, r = e & 15;
            if (m0 + m < M) {
                float v = 0.f;
#pragma unroll
                for (int k = 0; k < kSmallWarps; ++k) v += red[k][m][r];
                y[static_cast<size_t>(m0 + m) * N + 16 * t + r] = __float2half_rn(v);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------ dense product with fp16 output
// y[m][n] = sum_k x[m][k] * W[n][k]: fp16 operands, fp32 accumulation on mma.sync m16n8k16, fp16 output.  A block of
// four warps takes 64 tokens x 64 rows, warp w the tokens 16w .. 16w+15; fragments are read from global memory.
__global__ void __launch_bounds__(128) dense_f16_kernel(const __half* __restrict__ x, const __half* __restrict__ W, __half* __restrict__ y,
                                                        int M, int N, int K) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, c = lane & 3;
    const int m0 = blockIdx.y * 64 + 16 * warp, n0 = blockIdx.x * 64;
    const int ma = min(m0 + gq, M - 1), mb = min(m0 + gq + 8, M - 1);          // clamped for the loads, masked at the store
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
        const int o = k0 >> 1;
        const uint32_t a0 = __ldg(xa + o), a1 = __ldg(xb + o), a2 = __ldg(xa + o + 4), a3 = __ldg(xb + o + 4);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t b0 = __ldg(wr[t] + o), b1 = __ldg(wr[t] + o + 4);
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+f"(acc[t][0]), "+f"(acc[t][1]), "+f"(acc[t][2]), "+f"(acc[t][3])
                         : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int n = n0 + 8 * t + 2 * c;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int m = m0 + gq + 8 * h;
            if (m < M && n < N) *reinterpret_cast<__half2*>(y + static_cast<size_t>(m) * N + n) = __floats2half2_rn(acc[t][2 * h], acc[t][2 * h + 1]);
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
int small_packed_bytes(int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes) {
    SmallTable st;
    const int rc = make_small_table(N, K, g, bits_host, &st);
    if (rc != SLIM_OK) return rc;
    *out_bytes = static_cast<size_t>(g / 8) * N * st.prefix[st.G];
    return SLIM_OK;
}

int small_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes) {
    SmallTable st;
    const int rc = make_small_table(N, K, g, bits_host, &st);
    if (rc != SLIM_OK) return rc;
    // the batched path materialises the fp16 weights behind the status header
    *out_bytes = M > SLIM_GEMV_MAX_M ? 256 + static_cast<size_t>(N) * K * sizeof(__half) : 256;
    return SLIM_OK;
}

int small_pack(const uint8_t* codes, const uint8_t* bits_host, void* packed, int N, int K, int g, cudaStream_t s) {
    SmallTable st;
    const int rc = make_small_table(N, K, g, bits_host, &st);
    if (rc != SLIM_OK) return rc;
    if (N == 0 || K == 0) return SLIM_OK;
    if (codes == nullptr || packed == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(packed)) return SLIM_ERR_ALIGNMENT;
    const dim3 grid(static_cast<unsigned>((4ll * N * 4 + 255) / 256), static_cast<unsigned>(st.G));
    if (g == 32) pack_small_kernel<32><<<grid, 256, 0, s>>>(codes, static_cast<uint8_t*>(packed), N, K, st);
    else pack_small_kernel<64><<<grid, 256, 0, s>>>(codes, static_cast<uint8_t*>(packed), N, K, st);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

static int small_dequant_into(const void* packed, const SmallTable& st, const void* scales, const void* zeros, __half* W, int N, int K,
                              cudaStream_t s) {
    const unsigned grid = static_cast<unsigned>((static_cast<long long>(N) * (K / 8) + 255) / 256);
    if (st.T == 32)
        dequant_small_kernel<32><<<grid, 256, 0, s>>>(static_cast<const uint8_t*>(packed), static_cast<const __half*>(scales),
                                                       static_cast<const __half*>(zeros), W, N, K, st);
    else
        dequant_small_kernel<64><<<grid, 256, 0, s>>>(static_cast<const uint8_t*>(packed), static_cast<const __half*>(scales),
                                                       static_cast<const __half*>(zeros), W, N, K, st);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int small_dequant(const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros, void* W, int N, int K, int g,
                  cudaStream_t s) {
    SmallTable st;
    const int rc = make_small_table(N, K, g, bits_host, &st);
    if (rc != SLIM_OK) return rc;
    if (N == 0 || K == 0) return SLIM_OK;
    if (packed == nullptr || scales == nullptr || zeros == nullptr || W == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(zeros) || !aligned16(W)) return SLIM_ERR_ALIGNMENT;
    return small_dequant_into(packed, st, scales, zeros, static_cast<__half*>(W), N, K, s);
}

int small_linear(const void* x, const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros, void* y,
                 int M, int N, int K, int g, void* workspace, size_t workspace_bytes, cudaStream_t s) {
    SmallTable st;
    const int rc = make_small_table(N, K, g, bits_host, &st);
    if (rc != SLIM_OK) return rc;
    if (M == 0 || N == 0) return SLIM_OK;
    if (y == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(y)) return SLIM_ERR_ALIGNMENT;
    if (K == 0) {
        SLIM_CUDA_TRY(cudaMemsetAsync(y, 0, static_cast<size_t>(M) * N * sizeof(__half), s));
        return SLIM_OK;
    }
    if (x == nullptr || packed == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(packed) || !aligned16(scales) || !aligned16(zeros)) return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < 256) return SLIM_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
    const __half* xh = static_cast<const __half*>(x);
    const uint8_t* pk = static_cast<const uint8_t*>(packed);
    const __half* sc = static_cast<const __half*>(scales);
    const __half* zp = static_cast<const __half*>(zeros);
    __half* yh = static_cast<__half*>(y);
    if (M <= SLIM_GEMV_MAX_M) {
        const unsigned grid = static_cast<unsigned>(N / 16);
        if (g == 32) {
            if (M == 1) gemv_small_kernel<32, 1><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
            else if (M <= 4) gemv_small_kernel<32, 4><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
            else gemv_small_kernel<32, 8><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
        } else {
            if (M == 1) gemv_small_kernel<64, 1><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
            else if (M <= 4) gemv_small_kernel<64, 4><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
            else gemv_small_kernel<64, 8><<<grid, 32 * kSmallWarps, 0, s>>>(xh, pk, sc, zp, yh, M, N, K, st);
        }
        SLIM_CUDA_TRY(cudaGetLastError());
        return SLIM_OK;
    }
    if (workspace_bytes < 256 + static_cast<size_t>(N) * K * sizeof(__half)) return SLIM_ERR_WORKSPACE;
    __half* Wd = reinterpret_cast<__half*>(static_cast<uint8_t*>(workspace) + 256);
    const int rd = small_dequant_into(packed, st, scales, zeros, Wd, N, K, s);
    if (rd != SLIM_OK) return rd;
    const dim3 grid((N + 63) / 64, (M + 63) / 64);
    dense_f16_kernel<<<grid, 128, 0, s>>>(xh, Wd, yh, M, N, K);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim
