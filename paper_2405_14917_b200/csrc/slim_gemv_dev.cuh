// Device-side building blocks shared by the decode kernels (slim_mpq_gemv and the layer-set
// launch): PTX wrappers, the geometry of a slice word as a tensor-core operand, and the routine
// that puts one group of activations into B-fragment order.
#pragma once

#include "slim_common.cuh"

namespace slim {

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of a cluster barrier, for a rendezvous whose arrival can be signalled long before it is needed.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ float2 ld_cluster_f32x2(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(remote) : "memory");
    return v;
}

__device__ __forceinline__ void st_cluster_f32x2(uint32_t local_addr, uint32_t rank, float2 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1,%2};" ::"r"(remote), "f"(v.x), "f"(v.y) : "memory");
}

__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// D += A(f16, 16x16, row) * B(f16, 16x8, col), fp32 accumulate.
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y));
}

// ------------------------------------------------------------------------------------------ slice geometry
// A word of a width-w slice has nf = 32/w fields; pair p (0 <= p < nf/2) is fields p and p + nf/2,
// which sit 16 bits apart.  Pairs whose field ends above mantissa bit 9 are taken from the word
// shifted right by pair_shift(w).
__host__ __device__ constexpr int pair_shift(int w) { return w == 4 ? 8 : 10; }
__host__ __device__ constexpr bool pair_direct(int w, int p) { return w * p + w <= 10; }
// Bit position of pair p inside each half after the optional shift: the operand is v * 2^(pos-24).
__host__ __device__ constexpr int pair_pos(int w, int p) { return pair_direct(w, p) ? w * p : w * p - pair_shift(w); }

template <int W>
__device__ __forceinline__ uint32_t pair(uint32_t word, uint32_t sh, int p) {
    constexpr uint32_t kMask = 0x00010001u * ((1u << W) - 1u);
    return (pair_direct(W, p) ? word : sh) & (kMask << pair_pos(W, p));
}

template <int V> struct WidthTag { static constexpr int value = V; };
using W1 = WidthTag<1>;
using W2 = WidthTag<2>;
using W4 = WidthTag<4>;

// ------------------------------------------------------------------------------------------ activation staging
// Puts the 128 activations of one (token m, group) into B-fragment order for every slice of the
// group (lane = (mma mi, lane column cc) -> the four activations that meet that lane's two B
// registers) and returns the group's (sum_k x, 2^(24-S)) in lane 0.  xg: the group's 128 halves
// (shared or global); xs_slot0: first fragment slot of the group (shared or global).
__device__ __forceinline__ float2 stage_group(const __half* xg, uint8_t* xs_slot0, int b, int m, int M, int lane) {
    // 2^S lifts the group's largest |x| into [2^13, 2^14) (Inf/NaN: the top binade)
    const uint2 raw = *reinterpret_cast<const uint2*>(xg + 4 * lane);
    uint32_t mx = max(max(raw.x & 0x7fffu, (raw.x >> 16) & 0x7fffu), max(raw.y & 0x7fffu, (raw.y >> 16) & 0x7fffu));
    mx = __reduce_max_sync(0xffffffffu, mx);
    const int S = mx == 0 ? 0 : 28 - max(static_cast<int>(mx >> 10), 1);
    const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    float sum = (f01.x + f01.y) + (f23.x + f23.y);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const int cc = lane & 3, mi = lane >> 2;
    const int ns = slice_count(b);
    for (int s = 0; s < ns; ++s) {
        const int w = slice_w(b, s), lo = slice_lo(b, s);
        const int lg = w >> 1;                          // log2(w) for w in {1,2,4}
        const int nf = 32 >> lg;                        // fields per word; 8/w MMAs per unit
        const int u = mi >> (3 - lg), ii = mi & ((8 >> lg) - 1);
        const __half* xp = xg + 32 * cc + nf * u + 2 * ii;
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(xp));               // pairs 2ii, 2ii+1: first field
        const float2 g = __half22float2(*reinterpret_cast<const __half2*>(xp + (nf >> 1)));   // ... second field
        const float sc0 = __int_as_float((127 + S + lo - pair_pos(w, 2 * ii)) << 23);
        const float sc1 = __int_as_float((127 + S + lo - pair_pos(w, 2 * ii + 1)) << 23);
        const __half2 b0 = __floats2half2_rn(f.x * sc0, g.x * sc0);
        const __half2 b1 = __floats2half2_rn(f.y * sc1, g.y * sc1);
        *reinterpret_cast<uint2*>(xs_slot0 + (((static_cast<size_t>(s) * 8 + mi) * M + m) * 4 + cc) * 8) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&b0), *reinterpret_cast<const uint32_t*>(&b1));
    }
    return make_float2(sum, __int_as_float((127 + 24 - S) << 23));
}

}  // namespace slim
