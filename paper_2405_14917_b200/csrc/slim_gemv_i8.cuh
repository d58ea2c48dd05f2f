// Device code shared by the kernels of the single-token integer form of the decode path (slim_gemv_set.cu,
// slim_gemv_one.cu): bounded mbarrier waits and bulk copies, the staged layout of a group's activations, and the
// 8-bit digit form of x with its integer MMA.
#pragma once

#include "slim_gemv_dev.cuh"

namespace slim {

constexpr unsigned long long kSetWaitNs = 2000000000ull;      // limit of every device-side wait

// ------------------------------------------------------------------------------------------ mbarrier helpers
namespace sb {
__device__ __forceinline__ void init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrive by the lanes whose flag is set, as one predicated instruction (no divergent branch around it).
__device__ __forceinline__ void arrive_if(uint32_t bar, uint32_t flag) {
    asm volatile("{\n .reg .pred p;\n setp.ne.u32 p, %1, 0;\n @p mbarrier.arrive.shared::cta.b64 _, [%0];\n}\n" ::"r"(bar), "r"(flag) : "memory");
}
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up when `limit_ns` has passed or when another role has raised `abort`.
__device__ __forceinline__ bool wait_limit(uint32_t bar, uint32_t parity, volatile int* abort, unsigned long long limit_ns) {
    if (try_wait(bar, parity)) return true;
    const unsigned long long t0 = timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (try_wait(bar, parity)) return true;
        if (*abort != 0) return false;
        if (timer_ns() - t0 > limit_ns) { *abort = 1; return false; }
    }
}
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int* abort) {
    return wait_limit(bar, parity, abort, kSetWaitNs);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
}  // namespace sb

// ------------------------------------------------------------------------------------------ activation staging
// Byte offset of group j inside a layer's staged activations (pre3 = 3-bit groups before j).
// A record starts with (sum_k x, scale) per token, 8 bytes each: 128 bytes for up to 16 tokens, 8 M beyond.
__host__ __device__ constexpr int staged_header_bytes(int M) { return M > 16 ? 8 * M : 128; }
__host__ __device__ inline size_t staged_group_offset(int j, int pre3, int M) {
    return static_cast<size_t>(staged_header_bytes(M)) * static_cast<size_t>(j) + 256u * static_cast<size_t>(M) * static_cast<size_t>(j + pre3);
}
// ---- single-token sets: activations as signed 8-bit digits, the packed words as unsigned bytes ----------
// With one token seven of the eight MMA columns are free, and an integer MMA takes four codes per
// operand register where the f16 MMA takes two.  So for M = 1 the group's activations become the
// fixed-point X_k = rint(x_k 2^S) (|X| < 2^22: an fp16 value within a factor 2^11 of the group's largest
// is kept exactly), and every MMA's B operand holds the four signed base-256 digits of X_k 2^shift in
// columns 0..3 (columns 4..7 repeat them).  The A operand is the packed word ANDed with a byte-wise
// mask: byte value = field * 2^(w i) for the fields at position i of their byte (w = slice width), and
// shift = lo + Pc - w i <= 8 makes every product carry the same 2^Pc, so all positions and both slices
// of a 3-bit group add up in one set of integer accumulators (one per digit, each sum below 2^23: exact).
__host__ __device__ constexpr int i8_pc(int b) { return b == 1 ? 7 : (b == 4 ? 4 : 6); }
// Field position inside its byte that MMA mi meets in the A register half h, for a slice of width w.
__host__ __device__ constexpr int i8_pos(int w, int mi, int h) { return w == 1 ? mi + 4 * h : (w == 4 ? (mi & 1) : mi); }
// Column of the group that meets byte bb of the A register half h (k < 16 or k >= 16) of MMA mi, lane column c.
__device__ __forceinline__ int i8_column(int w, int mi, int h, int bb, int c) {
    return w == 2 ? 32 * c + 16 * h + 4 * bb + mi
         : w == 1 ? 32 * c + 8 * bb + mi + 4 * h
                  : 32 * c + 8 * (2 * (mi >> 1) + h) + 2 * bb + (mi & 1);
}
// Record of one group: (sum_k x, 2^(-S - Pc)) then, per slice, 4 MMAs x [4 digits][4 lanes] x 8 bytes.
__device__ __forceinline__ void stage_group_i8(const __half* xg, uint8_t* rec, int b, int lane, int* Xs) {
    const uint2 raw = *reinterpret_cast<const uint2*>(xg + 4 * lane);
    uint32_t mx = max(max(raw.x & 0x7fffu, (raw.x >> 16) & 0x7fffu), max(raw.y & 0x7fffu, (raw.y >> 16) & 0x7fffu));
    mx = __reduce_max_sync(0xffffffffu, mx);
    const int S = mx == 0 ? 0 : 36 - max(static_cast<int>(mx >> 10), 1);     // largest |x| 2^S in [2^21, 2^22)
    const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    float sum = (f01.x + f01.y) + (f23.x + f23.y);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float up = __int_as_float((127 + S) << 23);
    const int pc = i8_pc(b);
    Xs[4 * lane + 0] = __float2int_rn(f01.x * up);       // the group's fixed-point activations, once
    Xs[4 * lane + 1] = __float2int_rn(f01.y * up);
    Xs[4 * lane + 2] = __float2int_rn(f23.x * up);
    Xs[4 * lane + 3] = __float2int_rn(f23.y * up);
    __syncwarp();
    // lane = (MMA mi, lane column c, register half h): the four k-slots (bytes bb) of that B register, all four digits
    const int mi = lane >> 3, c = (lane >> 1) & 3, h = lane & 1;
    for (int sl = 0; sl < slice_count(b); ++sl) {
        const int w = slice_w(b, sl), lo = slice_lo(b, sl);
        // The MMA of a byte's top field position takes the packed word as it is, i.e. every field of the byte times
        // that position's digit; the other positions subtract it again.
        const int mi_top = w == 4 ? (mi | 1) : 3, h_top = w == 1 ? 1 : h;
        const int sh = lo + pc - w * i8_pos(w, mi, h), sh_top = lo + pc - w * i8_pos(w, mi_top, h_top);
        const bool is_top = mi == mi_top && h == h_top;
        uint32_t word[4] = {0u, 0u, 0u, 0u};               // digits 3 (highest) .. 0 of the four k-slots
        for (int bb = 0; bb < 4; ++bb) {
            int V = Xs[i8_column(w, mi, h, bb, c)] << sh;
            if (!is_top) V -= Xs[i8_column(w, mi_top, h_top, bb, c)] << sh_top;
            const int d0 = static_cast<int8_t>(V & 0xff), V1 = (V - d0) >> 8;      // |V| < 2^30 + 2^24
            const int d1 = static_cast<int8_t>(V1 & 0xff), V2 = (V1 - d1) >> 8;
            const int d2 = static_cast<int8_t>(V2 & 0xff), d3 = (V2 - d2) >> 8;    // |d3| <= 65
            word[0] |= static_cast<uint32_t>(d3 & 0xff) << (8 * bb);
            word[1] |= static_cast<uint32_t>(d2 & 0xff) << (8 * bb);
            word[2] |= static_cast<uint32_t>(d1 & 0xff) << (8 * bb);
            word[3] |= static_cast<uint32_t>(d0 & 0xff) << (8 * bb);
        }
#pragma unroll
        for (int n = 0; n < 4; ++n)
            *reinterpret_cast<uint32_t*>(rec + 128 + sl * 512 + mi * 128 + (n * 4 + c) * 8 + 4 * h) = word[n];
    }
    if (lane == 0) *reinterpret_cast<float2*>(rec) = make_float2(sum, __int_as_float((127 - S - pc) << 23));
}
// D (+)= A(u8, 16x32, row) * B(s8, 32x8, col), s32 accumulate.
__device__ __forceinline__ void mma_i8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y));
}
__device__ __forceinline__ void mma_i8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y), "r"(0));
}

}  // namespace slim
