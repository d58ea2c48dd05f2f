// slim_pack_weights and slim_dequant: integer bit shuffling between unpacked codes, the sliced
// bit-plane format and fp16 weights.  Both are one-off, memory-bound helpers.
#include "slim_common.cuh"

namespace slim {

// One thread per 32-bit word of the packed buffer.  grid.y = group, grid.x covers the 4*N*b words
// of the widest group; a word gathers 32/w consecutive codes of one row.
__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ codes, uint32_t* __restrict__ packed,
                                                   int N, int K, GroupTable gt) {
    const int j = blockIdx.y;
    const int b = gt.bits[j];
    const long long wi = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;  // word inside the group
    const long long words_in_group = 4ll * N * b;
    if (wi >= words_in_group) return;
    const int per_tile = 64 * b;
    const int t = static_cast<int>(wi / per_tile);
    const int rem = static_cast<int>(wi % per_tile);
    const int unit = rem >> 6;
    const int lane = (rem & 63) >> 1;
    const int half = rem & 1;
    const int s = (b == 3 && unit >= 2) ? 1 : 0;
    const int lo = slice_lo(b, s), w = slice_w(b, s), u = unit - slice_unit0(b, s);
    const int nf = 32 / w;
    const int c = lane & 3, gq = lane >> 2;
    const int row = 16 * t + 2 * gq + half;
    const int k0 = SLIM_GROUP * j + 32 * c + nf * u;
    const uint8_t* src = codes + static_cast<size_t>(row) * K + k0;
    const uint32_t mask = (1u << w) - 1u;
    uint32_t word = 0;
    // nf is 8, 16 or 32 and k0 is a multiple of nf: read 8 bytes at a time
    for (int f0 = 0; f0 < nf; f0 += 8) {
        const uint2 v = *reinterpret_cast<const uint2*>(src + f0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            word |= (((v.x >> (8 * i)) >> lo) & mask) << (w * (f0 + i));
            word |= (((v.y >> (8 * i)) >> lo) & mask) << (w * (f0 + 4 + i));
        }
    }
    packed[4ull * N * gt.prefix[j] + wi] = word;
}

// One thread per 8 consecutive columns of one row: reads one word per slice, writes 16 bytes.
__global__ void __launch_bounds__(256) dequant_kernel(const uint32_t* __restrict__ packed, const __half* __restrict__ scales,
                                                      const __half* __restrict__ zeros, __half* __restrict__ W,
                                                      int N, int K, GroupTable gt) {
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int per_row = K / 8;
    if (idx >= static_cast<long long>(N) * per_row) return;
    const int row = static_cast<int>(idx / per_row);
    const int k0 = static_cast<int>(idx % per_row) * 8;
    const int j = k0 / SLIM_GROUP, kk = k0 % SLIM_GROUP;
    const int b = gt.bits[j];
    const int t = row >> 4, r = row & 15, gq = r >> 1, half = r & 1, c = kk >> 5, rem = kk & 31;
    const uint32_t* grp = packed + 4ull * N * gt.prefix[j] + static_cast<size_t>(t) * 64 * b;
    uint32_t q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = 0;
    const int ns = slice_count(b);
    for (int s = 0; s < ns; ++s) {
        const int lo = slice_lo(b, s), w = slice_w(b, s), nf = 32 / w;
        const int u = rem / nf, f0 = rem % nf;
        const uint32_t word = grp[64 * (slice_unit0(b, s) + u) + 2 * (4 * gq + c) + half];
        const uint32_t mask = (1u << w) - 1u;
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] |= ((word >> (w * (f0 + i))) & mask) << lo;
    }
    const float sc = __half2float(scales[static_cast<size_t>(j >> gt.gshift) * N + row]);
    const float zp = __half2float(zeros[static_cast<size_t>(j >> gt.gshift) * N + row]);
    __align__(16) __half out[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) out[i] = __float2half_rn(__fmul_rn(sc, __fsub_rn(static_cast<float>(q[i]), zp)));
    *reinterpret_cast<uint4*>(W + static_cast<size_t>(row) * K + k0) = *reinterpret_cast<const uint4*>(out);
}

}  // namespace slim

extern "C" {

int slim_pack_weights(const uint8_t* codes, const uint8_t* bits_host, void* packed, int N, int K, int g, void* stream) {
    if (slim::is_small_group(g)) return slim::small_pack(codes, bits_host, packed, N, K, g, static_cast<cudaStream_t>(stream));
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (N == 0 || K == 0) return SLIM_OK;
    if (codes == nullptr || packed == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(codes) || !slim::aligned16(packed)) return SLIM_ERR_ALIGNMENT;
    const long long max_words = 4ll * N * 4;
    dim3 grid(static_cast<unsigned>((max_words + 255) / 256), static_cast<unsigned>(gt.G));
    slim::pack_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(codes, static_cast<uint32_t*>(packed), N, K, gt);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int slim_dequant(const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros, void* W,
                 int N, int K, int g, void* stream) {
    if (slim::is_small_group(g)) return slim::small_dequant(packed, bits_host, scales, zeros, W, N, K, g, static_cast<cudaStream_t>(stream));
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (N == 0 || K == 0) return SLIM_OK;
    if (packed == nullptr || scales == nullptr || zeros == nullptr || W == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(packed) || !slim::aligned16(scales) || !slim::aligned16(zeros) || !slim::aligned16(W))
        return SLIM_ERR_ALIGNMENT;
    const long long threads = static_cast<long long>(N) * (K / 8);
    const unsigned grid = static_cast<unsigned>((threads + 255) / 256);
    slim::dequant_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint32_t*>(packed), static_cast<const __half*>(scales), static_cast<const __half*>(zeros),
        static_cast<__half*>(W), N, K, gt);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // extern "C"
