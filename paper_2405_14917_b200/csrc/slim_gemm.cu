// slim_mpq_gemm: batched / prefill path (M > 16) of the mixed-precision linear layer, sm_100a.
//
// y^T = W-hat * x^T on the 5th-generation tensor cores, two CTAs (one cluster, two SMs) per MMA.
// The weight rows are the M dimension of the MMA (256 per pair, 128 per CTA), the tokens its N
// dimension (TOK = 128 or 256 per tile):
//
//  * A operand = dequantised weights, fp16, written by the dequant warps of each CTA straight
//    into that CTA's tensor memory with tcgen05.st (thread = weight row, 32-bit column = two
//    consecutive k); no shared memory round trip and no swizzled layout to reproduce.  One stage
//    = one group of 128 k.
//  * B operand = activations, x[tokens][k].  Each CTA brings HALF of the tile's tokens by TMA into
//    128-byte-swizzled K-major shared memory (two boxes of 64 k per group); the pair's MMA reads
//    both halves, so every SM pulls half the activation bytes a single-CTA tile would need and
//    the freed shared memory buys deeper pipelines.
//  * D = fp32 accumulator in tensor memory, 128 lanes x TOK columns per CTA; tcgen05.mma
//    cta_group::2 kind::f16 is issued by one thread of the leader CTA (cluster rank 0), eight
//    K=16 steps per group, and a multicast tcgen05.commit hands the stages back to both CTAs.
//  * Epilogue warps of each CTA read their D with tcgen05.ld and store y as fp16: a whole tile goes
//    through shared memory, 32 tokens x 32 rows per warp at a time, and out with one tensor store per
//    chunk (two buffers per warp: a chunk is written while the store of the one before reads its
//    buffer); the tensor map clips rows past N and tokens past M.
//
// Dequantisation: a code field is left in mantissa bits [6,10) of the half 1024; one HFMA2 with
// constants that hold the zero point turns it into q - z exactly for every zero point that is a
// multiple of 1/16 in [-16, 16) (all integer and half-integer zero points of Eq. 1 / Eq. 2), one
// HMUL2 applies the scale with a single rounding, so the operand equals the fp16 weight
// slim_dequant produces.  Other zero points are rounded (to the nearest 1/16 at worst).
//
// Warp roles (23 warps per CTA): warp 0 producer of activations (TMA); warp 1 MMA issuer in the
// leader / "my half of x has landed" relay in the other CTA, and tensor-memory allocator in both;
// warps 2-17 dequant, two sets of eight that take alternate groups; warps 18-21 epilogue; warp 22
// producer of packed slices, scales and zeros (bulk copies).  Persistent
// clusters walk the (token tile, 256-row block) tiles; every wait on an mbarrier or a flag is
// bounded and reports through the workspace status word instead of spinning forever, and no CTA
// leaves before its partner has stopped signalling it.
#include "slim_common.cuh"

#include <atomic>

#include <cuda.h>
#include <cstring>
#include <cmath>

namespace slim {

constexpr int kDqWarps = 16;                // dequant warps: sets of 8 that take the pipeline stages in turn
constexpr int kWarpEpi = 2 + kDqWarps;      // first of the four epilogue warps
constexpr int kWarpPacked = kWarpEpi + 4;   // producer of packed slices
constexpr int kGemmThreads = 32 * (kWarpPacked + 1);
constexpr int kRowsPerCta = 128;
constexpr int kRowsPerPair = 2 * kRowsPerCta;
constexpr int kGPS = 2;                     // groups per pipeline stage: one round of barriers serves this many
constexpr int kNS = 4 / kGPS;               // pipeline stages: a shared-memory slot of x + 64 tensor-memory columns of A per group
constexpr int kPStageBytes = 8192 + 512;    // 128 rows x 128 k x 4 bits, + scales + zeros
constexpr int kTmemCols = 512;
constexpr int kEpiCols = 16;                // accumulator columns (tokens) the epilogue handles at a time
constexpr int kYBox = 32;                   // tokens, and rows, of one output store
constexpr int kYBoxBytes = kYBox * kYBox * 2;
constexpr int kTmemAcol = 256;              // A stages start here; D occupies [0, TOK)
constexpr unsigned long long kGemmWaitNs = 2000000000ull;
constexpr unsigned int kGemmTryNs = 1000000u;     // suspend-time hint of one mbarrier.try_wait

struct GemmParams {
    const uint8_t* packed;
    const __half* scales;
    const __half* zeros;
    __half* y;
    unsigned int* status;
    unsigned int* flags;     // [grid]: "partial of this CTA is ready" (stream-K only; zero between launches)
    float* partials;         // [grid][4 epilogue warps][TOK][32 rows] fp32 (stream-K only)
    int M, N, K;
    int row_blocks, tok_tiles;   // 256-row blocks, TOK-token tiles
    int stream_k;            // 1: clusters take equal shares of (tile, group) units; 0: whole tiles
    GroupTable gt;
};

constexpr int kGemmWsFlags = 256;            // byte offset of the flags in the workspace
constexpr int kGemmMaxGrid = 256;
constexpr int kGemmWsPartials = kGemmWsFlags + 4 * kGemmMaxGrid;

// ------------------------------------------------------------------------------------------ PTX helpers
namespace g {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive on a barrier of any CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// One try: the thread may stay suspended for up to kGemmTryNs while the phase is pending (it wakes when the phase
// completes), so a waiting role re-issues its poll rarely; under the power cap that is worth 1.4 % of the M = 2048 rate.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kGemmTryNs) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Gives up when the limit passes or when another role has raised `abort`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort != 0) return false;
        if (global_timer_ns() - t0 > kGemmWaitNs) { *abort = 1; return false; }
    }
}
// The same by a whole warp: its lanes go on, or give up, together.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort));
}
// The same for a wait that is known to be long (a whole tile): one lane polls, with a pause
// between tries, so the waiting warp leaves the issue slots to the warps that work.
__device__ __forceinline__ bool mbar_wait_long(uint32_t bar, uint32_t parity, volatile int* abort) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0) {
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(bar, parity)) {
            __nanosleep(128);
            if (*abort != 0) { ok = false; break; }
            if (global_timer_ns() - t0 > kGemmWaitNs) { *abort = 1; ok = false; break; }
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (ok) ok = mbar_wait_warp(bar, parity, abort);  // every lane observes the completed phase itself
    return ok;
}
// After a failure: wait, for a millisecond at most, until the copies issued to a stage have landed.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    const unsigned long long t0 = global_timer_ns();
    while (!mbar_try_wait(bar, parity) && global_timer_ns() - t0 < 1000000ull) { }
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Tensor memory of the CTA pair: one warp of EACH CTA executes these together.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// When the pair's MMAs issued so far have completed, arrive on the barrier at this shared-memory
// offset in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor] over the CTA pair: 256 weight rows (128 from each
// CTA's tensor memory) x TOK tokens (half from each CTA's shared memory); fp16 in, fp32 accumulate.
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 lanes x 32 columns of 32-bit: thread = lane, register j = column j.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}
// 32 lanes x 16 columns
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// Shared memory -> global, tile of a tensor map (rows and columns past the tensor's extent are clipped).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest `N` stores of this thread have read their shared memory
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void sts_u16(uint32_t addr, uint16_t v) { asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory"); }
__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
// orders what this thread has observed through ordinary loads before the bulk copies it issues next
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
}  // namespace g

// ------------------------------------------------------------------------------------------ dequantisation
// Everything below works on one "c-word set": the slice words of one weight row that cover 32
// consecutive k, and produces the 16 tensor-memory columns (k, k+1 pairs) of those 32 weights.
//
// A code field q left at mantissa bit p under the exponent of 1024 is the half 1024 + q * 2^p, so
//     fma(v, 2^-p, -(2^(10-p) + z)) = q - z
// with no rounding whenever q - z is a half; the product with the scale then rounds once, like
// slim_dequant.  Positions 6..9 keep the constant 2^(10-p) + z below 32, where a half resolves
// 1/64.  One shifted copy of a slice word therefore serves every field that lands in bits [6,10):
// four 1-bit fields, two 2-bit fields or one 4-bit field; both halves of the word at once.
constexpr uint32_t kMagic1024 = 0x64006400u;            // half2(1024, 1024): ulp 1

__device__ __forceinline__ __half2 as_half2(uint32_t v) { return *reinterpret_cast<const __half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<const uint32_t*>(&h); }
// half2(2^e, 2^e), -14 <= e <= 15
__device__ __forceinline__ __half2 pow2_h2(int e) { return as_half2(0x00010001u * (static_cast<uint32_t>(e + 15) << 10)); }

struct DqRow {
    __half2 s;        // (s, s)
    __half2 add[4];   // -(constant of position i + z), see the decoders
};
__device__ __forceinline__ uint32_t lo_halves(uint32_t a, uint32_t b) { return g::prmt(a, b, 0x5410u); }
__device__ __forceinline__ uint32_t hi_halves(uint32_t a, uint32_t b) { return g::prmt(a, b, 0x7632u); }

// Logical shift, left if s > 0 (s is a constant after unrolling).
__device__ __forceinline__ uint32_t shift_to(uint32_t v, int s) { return s >= 0 ? v << s : v >> (-s); }

// Constants of a row for groups of B bits.  Position i of a copy holds a field at bit 6 + W*i
// (W = field width of the slice: 1, 2, 2, 4 for B = 1..4).  For B = 3 the third bit of pair f
// comes from a copy of the 1-bit slice at bit 6 + (f & 3) and enters through a second fma as
// 4 * bit + 2^(6 - (f & 3)); that constant is taken off in advance with the first one.
template <int B>
__device__ __forceinline__ void row_constants(__half s, __half z, DqRow& r) {
    r.s = __half2half2(s);
    const __half2 z2 = __half2half2(z);
    constexpr int W = B == 3 ? 2 : B;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float c = 0.f;
        if (B == 3) c = static_cast<float>(1 << (4 - 2 * (i & 1))) + static_cast<float>(1 << (6 - i));
        else if (W * i < 4) c = static_cast<float>(1 << (4 - W * i));
        r.add[i] = __hsub2(__float2half2_rn(-c), z2);
    }
}

// Fields of width W: F = 16/W pairs (f, f + F) per word; H[f] = (w[k0+f], w[k0+f+F]).  The word
// covers 2F consecutive k; its F columns are (H[2j].lo, H[2j+1].lo) for j < F/2 and the hi halves
// for the rest.  If HIGH, X carries a third code bit: bit f of its low/high half belongs to pair f.
template <int W, int F, bool HIGH>
__device__ __forceinline__ void decode_word(uint32_t word, uint32_t X, const DqRow& r, uint32_t* cols) {
    constexpr int PER = 4 / W;                                   // fields of one half served by one copy
    constexpr uint32_t kField = 0x00010001u * ((1u << W) - 1u);
    uint32_t H[F];
#pragma unroll
    for (int c = 0; c < F / PER; ++c) {
        const uint32_t copy = shift_to(word, 6 - 4 * c);
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int f = PER * c + i, pos = 6 + W * i;
            const uint32_t v = (copy & (kField << pos)) | kMagic1024;
            __half2 t = __hfma2(as_half2(v), pow2_h2(-pos), r.add[HIGH ? (f & 3) : i]);
            if (HIGH) {
                const int xpos = 6 + (f & 3);
                const uint32_t vb = (shift_to(X, 6 - 4 * (f >> 2)) & (0x00010001u << xpos)) | kMagic1024;
                t = __hfma2(as_half2(vb), pow2_h2(2 - xpos), t);
            }
            H[f] = as_u32(__hmul2(t, r.s));
        }
    }
#pragma unroll
    for (int j = 0; j < F / 2; ++j) {
        cols[j] = lo_halves(H[2 * j], H[2 * j + 1]);
        cols[F / 2 + j] = hi_halves(H[2 * j], H[2 * j + 1]);
    }
}

// words[u] = word of unit u for this row and this 32-k range.  cols[16].
template <int B>
__device__ __forceinline__ void decode_cword(const uint32_t (&words)[4], const DqRow& r, uint32_t* cols) {
    if constexpr (B == 1) {
        decode_word<1, 16, false>(words[0], 0u, r, cols);
    } else if constexpr (B == 2) {
        decode_word<2, 8, false>(words[0], 0u, r, cols);
        decode_word<2, 8, false>(words[1], 0u, r, cols + 8);
    } else if constexpr (B == 3) {
        // the 1-bit slice word holds k = bit index; bytes 2u and 2u+1 line up with the pairs of unit u
        decode_word<2, 8, true>(words[0], g::prmt(words[2], 0u, 0x4140u), r, cols);
        decode_word<2, 8, true>(words[1], g::prmt(words[2], 0u, 0x4342u), r, cols + 8);
    } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) decode_word<4, 4, false>(words[u], 0u, r, cols + 4 * u);
    }
}

// ------------------------------------------------------------------------------------------ kernel
template <int TOK> struct GemmCfg {
    static constexpr int HALF = TOK / 2;                     // tokens this CTA brings
    static constexpr int NP = 8;                             // shared-memory stages of packed slices
    static constexpr int XBOX = HALF * 128;                  // bytes of one TMA box: HALF rows x 64 k
    static constexpr int XSTAGE = 2 * XBOX;                  // one group: 128 k
    static constexpr int OFF_P = kNS * kGPS * XSTAGE;
    static constexpr int OFF_STAGE = OFF_P + NP * kPStageBytes;   // output staging: per epilogue warp two tiles of 32 tokens x 32 rows, fp16
    static constexpr int OFF_BAR = OFF_STAGE + 4 * 2 * kYBoxBytes;
    static constexpr int NPEERBAR = TOK / kEpiCols;         // per epilogue warp: one per 16-token piece of a peer's partial tile
    static constexpr int NBAR = 3 * kNS + 2 * NP + 2 + 4 * NPEERBAR;
    static constexpr int OFF_MISC = OFF_BAR + 8 * NBAR;      // tensor-memory base, abort flag
    static constexpr int SMEM = OFF_MISC + 16 + 1024;        // + slack to align the base to 1024
};

// Shared-memory matrix descriptor of a K-major, 128-byte-swizzled operand: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t sw128_kmajor_desc(uint32_t smem_addr) {
    return static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

template <int TOK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap y_map, const __grid_constant__ GemmParams p) {
    using C = GemmCfg<TOK>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (g::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (sbase - g::smem_u32(smem_raw));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = static_cast<int>(g::cluster_ctarank());     // 0 = leader of the pair
    const uint32_t bar0 = sbase + C::OFF_BAR;
    // Barriers of this CTA.  Stage s is ready for the MMA when `full(s)` of the LEADER completes:
    // 16 dequant warps of the pair have written A, the leader's half of x has landed (its TMA
    // signals that barrier directly) and the other CTA's relay has reported its half (which lands
    // on that CTA's `xl_full(s)`).  One multicast commit on `empty(s)` gives the stage back to the
    // x producers and dequant warps of both CTAs.
    auto xl_full = [&](int s) { return bar0 + 8 * s; };
    auto full = [&](int s) { return bar0 + 8 * (kNS + s); };
    auto empty = [&](int s) { return bar0 + 8 * (2 * kNS + s); };
    auto p_full = [&](int s) { return bar0 + 8 * (3 * kNS + s); };
    auto p_empty = [&](int s) { return bar0 + 8 * (3 * kNS + C::NP + s); };
    const uint32_t d_full = bar0 + 8 * (3 * kNS + 2 * C::NP);
    const uint32_t d_empty = d_full + 8;                 // leader's: 8 epilogue warps of the pair
    auto peer_full = [&](int q, int s) { return d_empty + 8 + 8 * (C::NPEERBAR * q + s); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_MISC);
    volatile int* abort = reinterpret_cast<volatile int*>(smem + C::OFF_MISC + 4);

    if (tid == 0) {
        for (int s = 0; s < kNS; ++s) { g::mbar_init(xl_full(s), 1); g::mbar_init(full(s), 18); g::mbar_init(empty(s), 1); }
        for (int s = 0; s < C::NP; ++s) { g::mbar_init(p_full(s), 1); g::mbar_init(p_empty(s), 8); }
        g::mbar_init(d_full, 1);
        g::mbar_init(d_empty, 8);
        for (int s = 0; s < 4 * C::NPEERBAR; ++s) g::mbar_init(peer_full(0, s), 1);
        *abort = 0;
        g::fence_barrier_init();
        g::fence_proxy_async();
    }
    if (warp == 1) {
        g::tmem_alloc(g::smem_u32(tmem_slot), kTmemCols);
        g::tmem_relinquish();
    }
    g::tc_fence_before();
    g::cluster_sync_all();          // both CTAs' barriers exist before either signals the other
    g::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int G = p.gt.G, N = p.N;
    const int total_tiles = p.row_blocks * p.tok_tiles;
    const int cl = blockIdx.x >> 1, ncl = gridDim.x >> 1;
    // This pair's contiguous range [u0, u1) of (tile, group) units, unit = tile * G + group,
    // tile = token tile * row_blocks + 256-row block.  Without stream-K the range is whole tiles.
    auto range_begin = [&](int c) -> long long {
        return p.stream_k ? (static_cast<long long>(c) * total_tiles * G) / ncl
                          : ((static_cast<long long>(c) * total_tiles) / ncl) * G;
    };
    const long long u0 = range_begin(cl), u1 = range_begin(cl + 1);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer of activations
        if (lane == 0) {
            int sx = 0;
            uint32_t phx = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok;) {
                const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
                const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
                u += ge - gb;
                const int m0 = (tile / p.row_blocks) * TOK + rank * C::HALF;     // my half of the token tile
                for (int j = gb; j < ge; j += kGPS) {
                    const int ng = min(kGPS, ge - j);                            // groups of this stage
                    if (!g::mbar_wait(empty(sx), phx ^ 1u, abort)) { ok = false; break; }
                    const uint32_t bar = rank == 0 ? full(sx) : xl_full(sx);
                    g::mbar_expect_tx(bar, ng * C::XSTAGE);
                    for (int i = 0; i < 2 * ng; ++i)                            // boxes of 64 k
                        g::tma_load_2d(sbase + sx * kGPS * C::XSTAGE + i * C::XBOX, &x_map, SLIM_GROUP * j + 64 * i, m0, bar);
                    if (++sx == kNS) { sx = 0; phx ^= 1u; }
                }
            }
            if (ok) {
                // every stage has been handed back: no commit of the leader is still on its way here
                for (int s = 0; s < kNS && ok; ++s) {
                    ok = g::mbar_wait(empty(sx), phx ^ 1u, abort);
                    if (++sx == kNS) { sx = 0; phx ^= 1u; }
                }
            } else {
                // leave no copy in flight: wait (bounded) for the last phase issued to every stage
                for (int s = 0; s < kNS; ++s) g::mbar_drain(rank == 0 ? full(s) : xl_full(s), s < sx ? phx : phx ^ 1u);
            }
        }
    } else if (warp == kWarpPacked) {
        // ------------------------------------------------------------------ producer of packed slices, scales, zeros
        // three lanes, one bulk copy each per group
        if (lane < 3) {
            int sp = 0;
            uint32_t php = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok;) {
                const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
                const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
                u += ge - gb;
                const int rb = 2 * (tile % p.row_blocks) + rank;                 // my 128-row block
                const int tiles_here = max(0, min(8, (N >> 4) - 8 * rb));
                const uint32_t sbytes = static_cast<uint32_t>(tiles_here) * 32u;
                const __half* sz = (lane == 1 ? p.scales : p.zeros) + kRowsPerCta * rb;
                for (int j = gb; j < ge; ++j) {
                    // the three lanes go on, or give up, together
                    if (!__all_sync(0x7u, g::mbar_wait(p_empty(sp), php ^ 1u, abort))) { ok = false; break; }
                    if (tiles_here > 0) {
                        const uint32_t b = p.gt.bits[j];
                        const uint32_t wbytes = static_cast<uint32_t>(tiles_here) * 256u * b;
                        const uint32_t dst = sbase + C::OFF_P + sp * kPStageBytes;
                        if (lane == 0) g::mbar_expect_tx(p_full(sp), wbytes + 2 * sbytes);
                        __syncwarp(0x7u);
                        if (lane == 0)
                            g::bulk_g2s(dst, p.packed + 16ull * N * p.gt.prefix[j] + static_cast<size_t>(8 * rb) * 256 * b, wbytes, p_full(sp));
                        else
                            g::bulk_g2s(dst + 8192 + 256 * (lane - 1), sz + static_cast<size_t>(j >> p.gt.gshift) * N, sbytes, p_full(sp));
                    } else if (lane == 0) {
                        g::mbar_arrive(p_full(sp));             // no row of mine exists: nothing to bring
                    }
                    if (++sp == C::NP) { sp = 0; php ^= 1u; }
                }
            }
            if (!ok)
                for (int s = 0; s < C::NP; ++s) g::mbar_drain(p_full(s), s < sp ? php : php ^ 1u);
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (leader)
            constexpr uint32_t idesc = (1u << 4) | (static_cast<uint32_t>(TOK >> 3) << 17) | (static_cast<uint32_t>(kRowsPerPair >> 4) << 24);
            int st = 0;
            uint32_t ph = 0, phd = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok;) {
                const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
                const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
                u += ge - gb;
                if (!g::mbar_wait(d_empty, phd ^ 1u, abort)) { ok = false; break; }   // both epilogues have drained D
                g::tc_fence_after();
                for (int j = gb; j < ge; j += kGPS) {
                    const int nk = 8 * min(kGPS, ge - j);                        // K = 16 steps of this stage
                    if (!g::mbar_wait(full(st), ph, abort)) { ok = false; break; }
                    g::tc_fence_after();
                    const uint32_t xs = sbase + st * kGPS * C::XSTAGE;
                    const uint32_t a_t = tmem + kTmemAcol + 64 * kGPS * st;
#pragma unroll
                    for (int ks = 0; ks < 8 * kGPS; ++ks) {
                        if (ks < nk) {
                            const uint64_t bdesc = sw128_kmajor_desc(xs + (ks >> 2) * C::XBOX + (ks & 3) * 32);
                            g::umma_f16_ts(tmem, a_t + 8 * ks, bdesc, idesc, (j > gb || ks != 0) ? 1u : 0u);
                        }
                    }
                    g::tc_commit_pair(empty(st));
                    if (++st == kNS) { st = 0; ph ^= 1u; }
                }
                if (ok) g::tc_commit_pair(d_full);
                phd ^= 1u;
            }
        } else if (lane == 0) {
            // -------------------------------------------------------------- relay (other CTA)
            // tells the leader that this CTA's half of a group's activations is in shared memory
            int sx = 0;
            uint32_t phx = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok;) {
                const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
                const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
                u += ge - gb;
                for (int j = gb; j < ge; j += kGPS) {
                    if (!g::mbar_wait(xl_full(sx), phx, abort)) { ok = false; break; }
                    g::mbar_arrive_cluster(g::map_to_cta(full(sx), 0));
                    if (++sx == kNS) { sx = 0; phx ^= 1u; }
                }
            }
        }
    } else if (warp < kWarpEpi) {
        // ------------------------------------------------------------------ dequant warps
        // Warp = (tensor-memory lane quarter, k half of the group, set).  The two sets take
        // alternate groups, so the fixed latencies of one group (barriers, shared-memory loads,
        // tensor-memory store) overlap with the arithmetic of the next.
        static_assert((kNS & (kNS - 1)) == 0 && (C::NP & (C::NP - 1)) == 0, "stage counters use masks");
        constexpr int kSets = kDqWarps / 8;
        const int q = warp & 3, kh = ((warp - 2) >> 2) & 1, set = (warp - 2) >> 3;
        const int r = 32 * q + lane;                            // row inside the block
        const int t = r >> 4, gq = (r & 15) >> 1, half = r & 1;
        bool ok = true;
        const uint32_t full_leader = g::map_to_cta(full(0), 0);
        int si = 0, gi = 0;                                     // running numbers of the stage and of the group in this CTA's range
        for (long long u = u0; u < u1 && ok;) {
            const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
            const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
            u += ge - gb;
            const int rb = 2 * (tile % p.row_blocks) + rank;
            const bool row_ok = kRowsPerCta * rb + r < N;
            for (int j = gb; j < ge && ok; j += kGPS, ++si) {
                const int ng = min(kGPS, ge - j);                                // groups of this stage
                const int g0 = gi;
                gi += ng;
                if (si % kSets != set) continue;
                const int sa = si & (kNS - 1);
                const uint32_t pha = (si / kNS) & 1;
#pragma unroll
                for (int i = 0; i < kGPS; ++i) {
                    if (i >= ng) break;
                    const int sp = (g0 + i) & (C::NP - 1);
                    const uint32_t php = ((g0 + i) / C::NP) & 1;
                    if (!g::mbar_wait_warp(p_full(sp), php, abort)) { ok = false; break; }
                    const int b = p.gt.bits[j + i];
                    const uint32_t stage = sbase + C::OFF_P + sp * kPStageBytes;
                    uint32_t w0[4] = {0, 0, 0, 0}, w1[4] = {0, 0, 0, 0};   // words of units 0..3 for the two 32-k ranges
                    __half sc = __float2half_rn(0.f), zp = sc;             // rows past N: weight 0
                    if (row_ok) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (u < b) {
                                const uint4 v = g::lds128(stage + t * 256 * b + 256 * u + 8 * (4 * gq + 2 * kh));
                                w0[u] = half ? v.y : v.x;
                                w1[u] = half ? v.w : v.z;
                            }
                        }
                        sc = *reinterpret_cast<const __half*>(smem + C::OFF_P + sp * kPStageBytes + 8192 + 2 * r);
                        zp = *reinterpret_cast<const __half*>(smem + C::OFF_P + sp * kPStageBytes + 8192 + 256 + 2 * r);
                    }
                    __syncwarp();
                    if (lane == 0) g::mbar_arrive(p_empty(sp));

                    const uint32_t a_t = tmem + (static_cast<uint32_t>(32 * q) << 16) + kTmemAcol + 64 * (kGPS * sa + i) + 32 * kh;
                    uint32_t cols[16];
                    DqRow row;
                    // first 32 k of my half, then (the stage's columns are free by now) the other 32
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t (&w)[4] = h == 0 ? w0 : w1;
                        switch (b) {
                            case 1: if (h == 0) row_constants<1>(sc, zp, row); decode_cword<1>(w, row, cols); break;
                            case 2: if (h == 0) row_constants<2>(sc, zp, row); decode_cword<2>(w, row, cols); break;
                            case 3: if (h == 0) row_constants<3>(sc, zp, row); decode_cword<3>(w, row, cols); break;
                            default: if (h == 0) row_constants<4>(sc, zp, row); decode_cword<4>(w, row, cols); break;
                        }
                        if (h == 0 && i == 0) {
                            if (!g::mbar_wait_warp(empty(sa), pha ^ 1u, abort)) { ok = false; break; }
                            g::tc_fence_after();
                        }
                        g::tmem_st16(a_t + 16 * h, cols);
                    }
                    if (!ok) break;
                }
                if (!ok) break;
                g::tc_wait_st();
                g::tc_fence_before();
                __syncwarp();
                if (lane == 0) g::mbar_arrive_cluster(full_leader + 8 * sa);
            }
        }
    } else if (warp < kWarpPacked) {
        // ------------------------------------------------------------------ epilogue warps
        // A segment that covers its whole tile is stored as fp16.  With stream-K a tile may be cut:
        // a pair whose segment does not start the tile leaves its fp32 partials in its CTAs'
        // workspace slots and raises their flags; the pair that starts the tile (it reaches that
        // segment last, the others reach theirs first) waits for those flags, adds the partials in
        // pair order and stores the tile.  Each CTA deals with the CTAs of the same rank, which
        // hold the same 128 rows.
        const int q = warp & 3;
        const int et = tid - 32 * kWarpEpi;                     // 0..127 among the epilogue threads
        uint32_t phd = 0;
        bool ok = true;
        const uint32_t d_empty_leader = g::map_to_cta(d_empty, 0);
        auto epi_sync = [] { asm volatile("bar.sync 1, 128;" ::: "memory"); };
        // barrier of the 128 epilogue threads that also ORs a flag: every thread gets the same answer, so the four
        // warps leave, or go on to the next named barrier, together
        auto epi_any = [](bool v) {
            uint32_t r;
            asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
                         : "=r"(r) : "r"(static_cast<uint32_t>(v)) : "memory");
            return r != 0;
        };
        for (long long u = u0; u < u1 && ok;) {
            const int tile = static_cast<int>(u / G), gb = static_cast<int>(u - static_cast<long long>(tile) * G);
            const int ge = static_cast<int>(min(static_cast<long long>(G), gb + (u1 - u)));
            u += ge - gb;
            const int rb = 2 * (tile % p.row_blocks) + rank, mt = tile / p.row_blocks;
            const int n = kRowsPerCta * rb + 32 * q + lane;
            const bool is_partial = gb > 0;
            // peers: the pairs after this one, up to the one that ends the tile (pairs with an empty
            // range take no part); peer k is CTA blockIdx.x + 2k
            int npeer = 0;
            if (!is_partial && ge < G) {
                for (int pc = cl + 1; pc < ncl; ++pc) {
                    ++npeer;
                    if (range_begin(pc + 1) >= static_cast<long long>(tile + 1) * G) break;
                }
            }
            // bit k-1: peer k has a segment (a cut leaves every pair at least eight groups and a tile has at most
            // SLIM_MAX_GROUPS of them, so there are fewer than 64 peers)
            unsigned long long act = 0ull;
            for (int k = 1; k <= npeer && k <= 64; ++k)
                if (range_begin(cl + k) < range_begin(cl + k + 1)) act |= 1ull << (k - 1);
            auto peer_active = [&](int k) { return ((act >> (k - 1)) & 1ull) != 0ull; };
            bool gave_up = !g::mbar_wait_long(d_full, phd, abort);
            gave_up = epi_any(gave_up);          // named barriers may follow, now or in a later unit: decide once for all
            if (gave_up) { ok = false; break; }
            g::tc_fence_after();
            if (npeer > 0) {
                // thread k-1 waits for peer k's flag; the barrier passes what each of them acquired on to everyone
                bool late = false;
                if (et < npeer && peer_active(et + 1)) {
                    volatile unsigned int* f = p.flags + blockIdx.x + 2 * (et + 1);
                    const unsigned long long t0 = g::global_timer_ns();
                    while (*f == 0u) {
                        if (*abort != 0 || g::global_timer_ns() - t0 > kGemmWaitNs) { *abort = 1; late = true; break; }
                    }
                    __threadfence();
                }
                if (epi_any(late)) { ok = false; break; }
            }
            // slot layout [epilogue warp][token][row of the warp]: the 16-token pieces of a warp are contiguous 2 KB
            float* my_slot = p.partials + static_cast<size_t>(blockIdx.x) * (TOK * kRowsPerCta) + q * (TOK * 32) + lane;
            const uint32_t stg = sbase + C::OFF_STAGE + q * 2 * kYBoxBytes + 2 * lane;    // my output staging, at my row
            const int n0 = kRowsPerCta * rb + 32 * q;
            bool bad = false;                    // a wait inside the owner's loop gave up
            if (!is_partial && npeer == 0) {
                // whole tile: 32 tokens at a time through shared memory, one tensor store per chunk; the
                // store of a chunk reads its buffer while the next chunk is written into the other one
#pragma unroll 1
                for (int cc = 0; cc < TOK / kYBox; ++cc) {
                    const uint32_t buf = stg + (cc & 1) * kYBoxBytes;
                    if (lane == 0) g::bulk_wait_read<1>();
                    __syncwarp();
                    uint32_t v[32];
                    g::tmem_ld32(tmem + (static_cast<uint32_t>(32 * q) << 16) + kYBox * cc, v);
                    g::tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const __half2 h = __floats2half2_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                        g::sts_u16(buf + (2 * i) * 2 * kYBox, __half_as_ushort(__low2half(h)));
                        g::sts_u16(buf + (2 * i + 1) * 2 * kYBox, __half_as_ushort(__high2half(h)));
                    }
                    g::fence_proxy_async();
                    __syncwarp();
                    const int m0 = mt * TOK + kYBox * cc;
                    if (lane == 0 && n0 < N && m0 < p.M) {
                        g::tma_store_2d(&y_map, n0, m0, buf - 2 * lane);
                        g::bulk_commit();
                    }
                }
            } else if (is_partial) {
#pragma unroll 1
                for (int cc = 0; cc < TOK / kEpiCols; ++cc) {
                    uint32_t v[kEpiCols];
                    g::tmem_ld16(tmem + (static_cast<uint32_t>(32 * q) << 16) + kEpiCols * cc, v);
                    g::tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < kEpiCols; ++i) my_slot[(kEpiCols * cc + i) * 32] = __uint_as_float(v[i]);
                }
            } else {
                // Owner of a cut tile.  This is the last segment of my range, so the activation stages are free (every
                // MMA that read them has completed): my quarter of them is a ring of 2 KB sub-slots into which lane 0
                // brings the peers' partials by bulk copies, one per (16-token piece, peer), a ring's worth ahead.
                // Piece by piece the peers are added in pair order, then the accumulator; two pieces make one
                // tensor store.
                constexpr int S = C::NPEERBAR;
                static_assert((S & (S - 1)) == 0 && S * 2048 * 4 <= C::OFF_P, "ring of the peers' partials");
                const int np_act = __popcll(act);
                const int J = S * np_act;
                // the active peer after peer k, going round
                auto next_peer = [&](int k) {
                    const unsigned long long above = k < 64 ? act >> k : 0ull;
                    return above != 0ull ? k + __ffsll(static_cast<long long>(above)) : __ffsll(static_cast<long long>(act));
                };
                const uint32_t ring = sbase + q * (S * 2048);
                const float* peer0 = p.partials + static_cast<size_t>(blockIdx.x) * (TOK * kRowsPerCta) + q * (TOK * 32);
                int j_iss = 0, k_iss = np_act > 0 ? next_peer(64) : 0, cc_iss = 0, a_iss = 0, j_con = 0;
                auto issue_next = [&]() {                        // job j_iss = (piece cc_iss, peer k_iss)
                    if (lane == 0) {
                        const uint32_t slot = j_iss & (S - 1);
                        g::mbar_expect_tx(peer_full(q, slot), 2048);
                        g::bulk_g2s(ring + slot * 2048, peer0 + static_cast<size_t>(2 * k_iss) * (TOK * kRowsPerCta) + cc_iss * 512, 2048,
                                    peer_full(q, slot));
                    }
                    ++j_iss;
                    k_iss = next_peer(k_iss);
                    if (++a_iss == np_act) { a_iss = 0; ++cc_iss; }
                };
                g::fence_proxy_async_all();                      // the flags were seen through ordinary loads
                while (j_iss < min(S, J)) issue_next();
#pragma unroll 1
                for (int cc = 0; cc < S && !bad; ++cc) {
                    float t[kEpiCols];
#pragma unroll
                    for (int i = 0; i < kEpiCols; ++i) t[i] = 0.f;
                    for (int a = 0; a < np_act; ++a) {
                        const uint32_t slot = j_con & (S - 1);
                        if (!g::mbar_wait_warp(peer_full(q, slot), (j_con / S) & 1, abort)) { bad = true; break; }
                        ++j_con;
#pragma unroll
                        for (int i = 0; i < kEpiCols; ++i) t[i] += g::lds_f32(ring + slot * 2048 + 128 * i + 4 * lane);
                        __syncwarp();
                        if (j_iss < J) issue_next();
                    }
                    if (bad) break;
                    uint32_t v[kEpiCols];
                    g::tmem_ld16(tmem + (static_cast<uint32_t>(32 * q) << 16) + kEpiCols * cc, v);
                    g::tc_wait_ld();
                    const uint32_t buf = stg + ((cc >> 1) & 1) * kYBoxBytes + (cc & 1) * (kEpiCols * 2 * kYBox);
                    if ((cc & 1) == 0) {
                        if (lane == 0) g::bulk_wait_read<1>();
                        __syncwarp();
                    }
#pragma unroll
                    for (int i = 0; i < kEpiCols / 2; ++i) {
                        const __half2 h = __floats2half2_rn(__uint_as_float(v[2 * i]) + t[2 * i], __uint_as_float(v[2 * i + 1]) + t[2 * i + 1]);
                        g::sts_u16(buf + (2 * i) * 2 * kYBox, __half_as_ushort(__low2half(h)));
                        g::sts_u16(buf + (2 * i + 1) * 2 * kYBox, __half_as_ushort(__high2half(h)));
                    }
                    if (cc & 1) {
                        g::fence_proxy_async();
                        __syncwarp();
                        const int m0 = mt * TOK + kEpiCols * (cc - 1);
                        if (lane == 0 && n0 < N && m0 < p.M) {
                            g::tma_store_2d(&y_map, n0, m0, stg - 2 * lane + ((cc >> 1) & 1) * kYBoxBytes);
                            g::bulk_commit();
                        }
                    }
                }
                if (bad)                                         // leave no copy in flight
                    for (int j = j_con; j < j_iss; ++j) g::mbar_drain(peer_full(q, j & (S - 1)), (j / S) & 1);
            }
            g::tc_fence_before();
            __syncwarp();
            if (lane == 0) g::mbar_arrive_cluster(d_empty_leader);
            phd ^= 1u;
            if (is_partial) {
                __threadfence();
                epi_sync();
                if (et == 0) { __threadfence(); *(volatile unsigned int*)(p.flags + blockIdx.x) = 1u; }
            } else if (npeer > 0) {
                if (epi_any(bad)) { ok = false; break; }        // everyone has read the peers' slots
                if (et < npeer) p.flags[blockIdx.x + 2 * (1 + et)] = 0u;   // ready for the next launch (unused ones are 0 already)
            }
        }
        if (lane == 0) g::bulk_wait_all();                      // my stores have been written
    }

    // nobody leaves, and the pair's tensor memory stays, until both CTAs are through
    g::tc_fence_before();
    g::cluster_sync_all();
    if (tid == 0 && *abort != 0) atomicOr(p.status, 1u);
    if (warp == 1) {
        g::tc_fence_after();
        g::tmem_dealloc(tmem, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Tensor map of x [M][K] fp16: boxes of 64 k x `rows` tokens, 128-byte swizzle, rows past M read as 0.
static bool make_x_map(CUtensorMap* map, const void* x, int M, int K, int rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(M)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * sizeof(__half)};
    const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(rows)};
    const cuuint32_t estr[2] = {1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of y [M][N] fp16 for the epilogue's stores: boxes of 32 rows of W x 32 tokens, no swizzle.
static bool make_y_map(CUtensorMap* map, void* y, int M, int N) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(N) * sizeof(__half)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kYBox), static_cast<cuuint32_t>(kYBox)};
    const cuuint32_t estr[2] = {1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int gemm_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// CTA pairs that can be resident at once (the stream-K hand-over needs all of them running).
template <int TOK>
static int max_resident_pairs() {
    static std::atomic<int> cached[64];       // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        if (cudaFuncSetAttribute(gemm_kernel<TOK>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<TOK>::SMEM) != cudaSuccess) return 0;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(2 * gemm_sm_count(), 1, 1);
        cfg.blockDim = dim3(kGemmThreads, 1, 1);
        cfg.dynamicSmemBytes = GemmCfg<TOK>::SMEM;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_kernel<TOK>, &cfg) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            return 0;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

// Launch shape shared by the entry point and the workspace query.  Stream-K (equal shares of
// (tile, group) units per CTA pair, partial tiles combined through the workspace) is used when it
// is predicted to beat whole tiles, whose last wave may leave most SMs idle.
struct GemmPlan {
    int tok, row_blocks, tok_tiles, grid, stream_k;
    size_t workspace_bytes;
};
static GemmPlan plan_gemm(int M, int N, int G) {
    GemmPlan pl;
    pl.tok = M <= 128 ? 128 : 256;
    pl.row_blocks = (N + kRowsPerPair - 1) / kRowsPerPair;
    pl.tok_tiles = (M + pl.tok - 1) / pl.tok;
    const int tiles = pl.row_blocks * pl.tok_tiles;
    int pairs = gemm_sm_count() / 2;
    const int resident = pl.tok == 128 ? max_resident_pairs<128>() : max_resident_pairs<256>();
    if (resident > 0 && pairs > resident) pairs = resident;
    if (pairs > kGemmMaxGrid / 2) pairs = kGemmMaxGrid / 2;
    if (pairs < 1) pairs = 1;
    const int npairs = tiles < pairs ? tiles : pairs;
    const int waves = (tiles + pairs - 1) / pairs;
    pl.grid = 2 * npairs;
    pl.stream_k = 0;
    // Time in units of one group.  Whole tiles take waves * G.  Equal shares of the (tile, group) units over P
    // pairs take units / P plus the hand-over of the cut tiles: a dozen groups' worth when a tile has one peer
    // (drains, flags, one partial tile brought in and added), with more peers seven more per peer at 256 tokens
    // and three and a half at 128 (measured: graph-replayed timings of nine layer shapes at M = 32 ... 2048 with
    // either schedule).  P is every resident pair, or, for a layer with few tiles, two, three or four pairs per
    // tile: the cuts then fall on the same groups in every tile and a tile has one, two or three peers, where
    // equal shares over all pairs would give it more.
    const long long units = static_cast<long long>(tiles) * G;
    const double per_peer = pl.tok == 256 ? 7.0 : 3.5;
    double best = 0.95 * static_cast<double>(waves) * G;
    for (int k = 1; k <= 4 && resident > 0; ++k) {
        const int P = k == 1 ? pairs : k * tiles;
        if (P > pairs || units < 8ll * P) continue;
        const double share = static_cast<double>(units) / P;
        const double peers = k == 1 ? ceil(static_cast<double>(G) / share) : static_cast<double>(k - 1);
        const double cost = share + 12.0 + (peers > 1.0 ? per_peer * peers : 0.0);
        if (cost < best) {
            best = cost;
            pl.stream_k = 1;
            pl.grid = 2 * P;
        }
    }
    pl.workspace_bytes = pl.stream_k ? kGemmWsPartials + static_cast<size_t>(pl.grid) * pl.tok * kRowsPerCta * sizeof(float) : 256;
    return pl;
}
size_t gemm_workspace_bytes(int M, int N, int G) { return plan_gemm(M, N, G).workspace_bytes; }

template <int TOK>
static cudaError_t launch_gemm(const CUtensorMap& map, const CUtensorMap& ymap, const GemmParams& prm, int grid, cudaStream_t stream) {
    static std::atomic<bool> attr_set[64];    // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemm_kernel<TOK>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<TOK>::SMEM);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    gemm_kernel<TOK><<<grid, kGemmThreads, GemmCfg<TOK>::SMEM, stream>>>(map, ymap, prm);   // clusters of 2: see the kernel
    return cudaGetLastError();
}

}  // namespace slim

extern "C" int slim_mpq_gemm(const void* x, const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros,
                             void* y, int M, int N, int K, int g, void* workspace, size_t workspace_bytes, void* stream) {
    if (M < 0) return SLIM_ERR_INVALID_ARG;
    if (M > 0 && M <= SLIM_GEMV_MAX_M) return SLIM_ERR_INVALID_ARG;     // the decode path serves these
    if (slim::is_small_group(g))
        return slim::small_linear(x, packed, bits_host, scales, zeros, y, M, N, K, g, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (M == 0 || N == 0) return SLIM_OK;
    if (y == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(y)) return SLIM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (K == 0) {
        SLIM_CUDA_TRY(cudaMemsetAsync(y, 0, static_cast<size_t>(M) * N * sizeof(__half), s));
        return SLIM_OK;
    }
    if (x == nullptr || packed == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(x) || !slim::aligned16(packed) || !slim::aligned16(scales) || !slim::aligned16(zeros))
        return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < 256) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;

    slim::GemmPlan pl = slim::plan_gemm(M, N, gt.G);
    if (pl.stream_k && workspace_bytes < pl.workspace_bytes) {   // small workspace: whole tiles, no scratch
        pl.stream_k = 0;
        const int tiles = pl.row_blocks * pl.tok_tiles;
        if (pl.grid > 2 * tiles) pl.grid = 2 * tiles;
    }
    const int tok = pl.tok;
    CUtensorMap map;
    CUtensorMap ymap;
    if (!slim::make_x_map(&map, x, M, K, tok / 2) || !slim::make_y_map(&ymap, y, M, N)) {
        slim::set_cuda_error(cudaErrorUnknown);
        return SLIM_ERR_CUDA;
    }
    slim::GemmParams prm;
    memset(&prm, 0, sizeof prm);
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.zeros = static_cast<const __half*>(zeros);
    prm.y = static_cast<__half*>(y);
    prm.status = static_cast<unsigned int*>(workspace);
    prm.M = M; prm.N = N; prm.K = K;
    prm.flags = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(workspace) + slim::kGemmWsFlags);
    prm.partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + slim::kGemmWsPartials);
    prm.row_blocks = pl.row_blocks;
    prm.tok_tiles = pl.tok_tiles;
    prm.stream_k = pl.stream_k;
    prm.gt = gt;
    const cudaError_t e = tok == 128 ? slim::launch_gemm<128>(map, ymap, prm, pl.grid, s) : slim::launch_gemm<256>(map, ymap, prm, pl.grid, s);
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

// ------------------------------------------------------------------------------------------ no-allocation variant
// Built-in scratch for slim_mpq_gemm_static: the control words plus one fp32 partial tile per CTA
// of a 148-SM device.  It lives in every GPU that loads the library, for the life of the process.
static_assert(SLIM_STATIC_SCRATCH_MAX == slim::kGemmWsPartials + 148 * 256 * slim::kRowsPerCta * 4, "scratch size");
static __device__ __align__(256) unsigned char g_static_scratch[SLIM_STATIC_SCRATCH_MAX];

extern "C" int slim_mpq_gemm_static(const void* x, const void* packed, const uint8_t* bits_host, const void* scales,
                                    const void* zeros, void* y, int M, int N, int K, int g,
                                    unsigned int* status_out, void* stream) {
    if (M < 0 || (M > 0 && M <= SLIM_GEMV_MAX_M)) return SLIM_ERR_INVALID_ARG;
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (status_out != nullptr && (reinterpret_cast<uintptr_t>(status_out) & 3u) != 0) return SLIM_ERR_ALIGNMENT;
    if (M == 0 || N == 0 || K == 0) {  // nothing needs scratch: the ordinary entry point handles these
        const int rc0 = slim_mpq_gemm(x, packed, bits_host, scales, zeros, y, M, N, K, g, nullptr, 0, stream);
        if (rc0 == SLIM_OK && status_out != nullptr)
            SLIM_CUDA_TRY(cudaMemsetAsync(status_out, 0, sizeof(unsigned int), static_cast<cudaStream_t>(stream)));
        return rc0;
    }
    // what this shape wants on this device; more than the array holds is refused, never truncated
    if (slim::gemm_workspace_bytes(M, N, gt.G) > static_cast<size_t>(SLIM_STATIC_SCRATCH_MAX)) return SLIM_ERR_STATIC_SCRATCH;

    // Device address of the array, looked up once per device (the array's name is only a
    // host-side handle here and must not be handed to a kernel).
    static std::atomic<void*> scratch_ptr[64];   // zero-initialised; the look-up is idempotent
    int dev = 0;
    SLIM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SLIM_ERR_UNSUPPORTED;
    if (scratch_ptr[dev].load() == nullptr) {
        void* ptr = nullptr;
        SLIM_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        scratch_ptr[dev].store(ptr);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps what the last call left: the status word and the flags must start at zero
    SLIM_CUDA_TRY(cudaMemsetAsync(scratch_ptr[dev].load(), 0, slim::kGemmWsPartials, s));
    const int rc = slim_mpq_gemm(x, packed, bits_host, scales, zeros, y, M, N, K, g, scratch_ptr[dev].load(),
                                 SLIM_STATIC_SCRATCH_MAX, stream);
    if (rc != SLIM_OK) return rc;
    if (status_out != nullptr)
        SLIM_CUDA_TRY(cudaMemcpyAsync(status_out, scratch_ptr[dev].load(), sizeof(unsigned int), cudaMemcpyDeviceToDevice, s));
    return SLIM_OK;
}
