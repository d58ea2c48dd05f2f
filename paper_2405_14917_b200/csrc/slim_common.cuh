// Shared host-side helpers of the CUDA library: argument validation, the group table that
// every kernel receives by value, and the last-CUDA-error slot.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/slim.h"

namespace slim {

// Group table passed by value in kernel parameters (the paper's "additional array" of group
// bit-widths plus the "cumulative calculations" that give each group's start, App. B.2).
struct GroupTable {
    int G;                                 // K-tiles of 128 columns
    int gshift;                            // a group is 2^gshift consecutive K-tiles (g = 128, 256, 512): tile j belongs to
                                           // group j >> gshift, whose scale and zero-point rows it shares
    uint16_t prefix[SLIM_MAX_GROUPS + 1];  // prefix[j] = b_0 + ... + b_{j-1} over the K-tiles
    uint8_t bits[SLIM_MAX_GROUPS];         // bit-width of every K-tile
};

void set_cuda_error(cudaError_t e);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Scratch bytes slim_mpq_gemm wants for (M, N) on the current device (256 when it needs none).
size_t gemm_workspace_bytes(int M, int N, int G);

// slim_mpq_gemv sends large layers through the layer-set kernels: workspace bytes that takes (0: this shape stays on the
// per-layer kernel), and the call itself (SLIM_OK, a negative status, or 1 if not taken).
size_t gemv_route_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, const GroupTable& gt);
int gemv_route(const void* x, const void* packed, const uint8_t* bits_host, const GroupTable& gt, const void* scales, const void* zeros,
               void* y, int M, int N, int K, int g, void* workspace, size_t workspace_bytes, cudaStream_t stream);

// slim_mpq_gemv sends single-token layers whose K fits a CTA's shared memory to a kernel of their own (slim_gemv_one.cu):
// SLIM_OK, a negative status, or 1 if not taken.
int gemv_one(const void* x, const void* packed, const GroupTable& gt, const void* scales, const void* zeros, void* y,
             int M, int N, int K, void* workspace, cudaStream_t stream);

// A set of single-token layers as one resident launch of that kernel (small sets: q/k/v, gate/up).  one_set_plan decides
// (SLIM_OK: taken, descriptors written into the plan buffer; 1: not taken; negative: error), one_set_launch runs it.
struct OneSetPlan {
    int pairs, cluster, grid;
    size_t smem;
};
constexpr size_t kOneSetPlanHeader = 4096;       // CTA ranges of the layers, then the descriptors
int one_set_plan(const slim_layer* layers, int n_layers, int g, void* plan, size_t plan_bytes, cudaStream_t stream, OneSetPlan* out);
int one_set_launch(const OneSetPlan& pl, const void* plan, int n_layers, void* workspace, cudaStream_t stream);

// Validates shape arguments and fills the table, for group sizes of 128, 256 and 512 columns (bits_host has K / g
// entries).  Returns SLIM_OK or an error status; SLIM_ERR_UNSUPPORTED for the group sizes 32 and 64, which have
// kernels of their own (is_small_group).
int make_group_table(int N, int K, int g, const uint8_t* bits_host, GroupTable* out);
inline bool is_small_group(int g) { return g == 32 || g == 64; }

// Group sizes of 32 and 64 columns (slim_small_group.cu): same contracts as the entry points that call them.
int small_packed_bytes(int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes);
int small_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes);
int small_pack(const uint8_t* codes, const uint8_t* bits_host, void* packed, int N, int K, int g, cudaStream_t s);
int small_dequant(const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros, void* W, int N, int K, int g,
                  cudaStream_t s);
int small_linear(const void* x, const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros, void* y,
                 int M, int N, int K, int g, void* workspace, size_t workspace_bytes, cudaStream_t s);

#define SLIM_CUDA_TRY(expr)                                    \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) {                               \
            ::slim::set_cuda_error(_e);                        \
            return SLIM_ERR_CUDA;                              \
        }                                                      \
    } while (0)

// Slice table of a b-bit code: number of slices, and (lo, w, first unit) of each.
__host__ __device__ inline int slice_count(int b) { return b == 3 ? 2 : 1; }
__host__ __device__ inline int slice_lo(int b, int s) { return (b == 3 && s == 1) ? 2 : 0; }
__host__ __device__ inline int slice_w(int b, int s) { return b == 3 ? (s == 0 ? 2 : 1) : b; }
__host__ __device__ inline int slice_unit0(int b, int s) { return (b == 3 && s == 1) ? 2 : 0; }

}  // namespace slim
