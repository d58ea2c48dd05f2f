// slim_mpq_gemv: decode path (1 <= M <= 16) of the mixed-precision linear layer, sm_100a.
//
// The kernel streams the packed slices exactly once (HBM-bound) and does the dot products on
// the tensor cores without ever materialising fp16 weights:
//
//  * A operand = raw code slices.  A byte whose low nibble holds a code field v (v <= 15) and
//    whose high nibble is zero is, read as FP8 E4M3, exactly v * 2^-9 (subnormals and the first
//    binade are linear in the bit pattern).  So one AND isolates the same field of four weights
//    and yields four ready-to-use E4M3 operands; fields in the high nibble need one shift first.
//    The position of a field inside the nibble (bit 0..3) multiplies its value by a power of two.
//  * B operand = activations.  Each fp16 x[m][k] is split exactly into four E5M2 pieces (3
//    significant bits each, 4 x 3 >= 11); the four pieces of a token occupy four columns of the
//    m16n8k32 tile, so one n-tile serves two tokens.  While staging, each piece is multiplied by
//    the power of two that undoes the field position and slice offset of the weight it will meet,
//    and by a per-token power of two 2^S that centres the token's range in E5M2.
//  * mma.sync.m16n8k32.e4m3.e5m2 accumulates the exact products in fp32.  Per (row, group) the
//    group partial D is folded as acc += s * (D - z * sum_k x_k), which is s * sum_k x_k (q_k - z).
//  * At the end the piece columns of a token are added and scaled by 2^(9-S).
//
// Work split: grid = (row blocks of 128*T rows) x (SK contiguous group ranges).  Each of the 8
// warps of a CTA owns T 16-row tiles and walks the CTA's group range; for one group its T tiles
// are one contiguous run of the packed buffer, fetched with one bulk async copy (plus two small
// ones for scales and zeros) into a warp-private ring of stages guarded by mbarriers.  Split-K
// partials go to the workspace; the last CTA of a row block (atomic ticket) adds them in a fixed
// order, so results are deterministic.
//
// The kernel is launched with programmatic stream serialisation: it issues its first weight
// copies, lets the next kernel start, and only then waits for the previous kernel before it
// touches x, y or the workspace.  Back-to-back layers therefore overlap their weight streams.
#include "slim_common.cuh"

#include <cstring>

namespace slim {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxSplit = 64;
constexpr int kMaxStages = 8;
constexpr int kWsHeader = 256;              // status word + padding
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct GemvParams {
    const __half* x;
    const uint8_t* packed;
    const __half* scales;
    const __half* zeros;
    __half* y;
    float* partials;        // [SK][M][N] fp32 (workspace)
    unsigned int* counters; // [row blocks] (workspace)
    unsigned int* status;   // workspace status word
    int M, N, K;
    int SK;
    int nstage;
    int stage_bytes;        // bytes of one ring stage (weights of T tiles at the widest group + scales + zeros)
    int w_stage_bytes;      // offset of the scales inside a stage
    int max_groups;         // widest group range of any split (sizes the x staging area)
    int max_slots;          // most slices in any group range
    uint16_t kbegin[kMaxSplit + 1];
    GroupTable gt;
};

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after kWaitLimitNs and reports false (the caller flags the error and
// stops consuming; nothing ever spins without a limit).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kWaitLimitNs) return false;
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// D += A(e4m3, 16x32) * B(e5m2, 32x8), fp32 accumulate.
__device__ __forceinline__ void mma_e4m3_e5m2(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e5m2.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y));
}

// ------------------------------------------------------------------------------------------ slice geometry
// Field p (0 .. 8/W-1) of every byte of a slice word, isolated in the low nibble of its byte.
// `sh` is the word shifted right by 4 (computed once per word by the caller).
template <int W>
__device__ __forceinline__ uint32_t field(uint32_t word, uint32_t sh, int p) {
    constexpr int kPerNibble = 4 / W;                     // fields that fit in one nibble
    constexpr uint32_t kMask = 0x01010101u * ((1u << W) - 1u);
    const uint32_t src = (p < kPerNibble) ? word : sh;
    return src & (kMask << (W * (p % kPerNibble)));
}
// Bit position of field p inside its nibble after the optional shift: its value is scaled by 2^pos.
__host__ __device__ __forceinline__ int field_pos(int w, int p) { return w * (p % (4 / w)); }

template <int V> struct WidthTag { static constexpr int value = V; };
using W1 = WidthTag<1>;
using W2 = WidthTag<2>;
using W4 = WidthTag<4>;

// ------------------------------------------------------------------------------------------ shared memory map
struct SmemMap {
    uint32_t mbar;     // kWarps * nstage * 8
    uint32_t sexp;     // int[16]: per-token power-of-two exponent S
    uint32_t xslot;    // uint16[max_groups + 1]: first staging slot of each group of the range
    uint32_t sx;       // float[max_groups][8*NT]: 2^(S-9) * sum_k x (piece-0 columns only)
    uint32_t xraw;     // half[M][max_groups*128]
    uint32_t xs;       // [slots][4 mma][NT][32 lanes][8 B]
    uint32_t ring;     // kWarps * nstage * stage_bytes
    uint32_t total;
};
__host__ __device__ inline uint32_t align_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }
__host__ __device__ inline SmemMap make_smem_map(int NT, int M, int nstage, int stage_bytes, int max_groups, int max_slots) {
    SmemMap m;
    uint32_t o = 0;
    m.mbar = o;  o += kWarps * kMaxStages * 8;
    m.sexp = o;  o += 64;
    m.xslot = o; o += align_up(2 * (max_groups + 1), 16);
    m.sx = o;    o += align_up(4 * max_groups * 8 * NT, 16);
    m.xraw = o;  o += align_up(2 * M * max_groups * SLIM_GROUP, 16);
    o = align_up(o, 128);
    m.xs = o;    o += static_cast<uint32_t>(max_slots) * 4 * NT * 256;
    o = align_up(o, 128);
    m.ring = o;  o += static_cast<uint32_t>(kWarps) * nstage * stage_bytes;
    m.total = o;
    return m;
}

// ------------------------------------------------------------------------------------------ kernel
template <int NT, int T>
__global__ void __launch_bounds__(kThreads, 2) gemv_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const SmemMap sm = make_smem_map(NT, p.M, p.nstage, p.stage_bytes, p.max_groups, p.max_slots);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, c = lane & 3;
    const int rb = blockIdx.x, ks = blockIdx.y;
    const int N = p.N, M = p.M;
    const int g0 = p.kbegin[ks], g1 = p.kbegin[ks + 1];
    const int ng = g1 - g0;

    const int tiles_total = N >> 4;
    const int tile0 = (rb * kWarps + warp) * T;
    const int tw = min(T, tiles_total - tile0);            // tiles this warp owns (<= 0: none)
    const bool active = tw > 0;

    const uint32_t my_bar = sbase + sm.mbar + warp * kMaxStages * 8;
    const uint32_t my_ring = sbase + sm.ring + static_cast<uint32_t>(warp) * p.nstage * p.stage_bytes;

    // ---- producer side: one chunk = (this warp's tiles, one group): weights, scales, zeros
    auto issue_chunk = [&](int it) {
        const int j = g0 + it;
        const int b = p.gt.bits[j];
        const int st = it % p.nstage;
        const uint32_t bar = my_bar + st * 8;
        const uint32_t dst = my_ring + st * p.stage_bytes;
        const uint32_t wbytes = static_cast<uint32_t>(tw) * 256u * b;
        const uint32_t sbytes = static_cast<uint32_t>(tw) * 32u;
        mbar_expect_tx(bar, wbytes + 2 * sbytes);
        bulk_g2s(dst, p.packed + 16ull * N * p.gt.prefix[j] + static_cast<size_t>(tile0) * 256 * b, wbytes, bar);
        bulk_g2s(dst + p.w_stage_bytes, p.scales + static_cast<size_t>(j) * N + 16 * tile0, sbytes, bar);
        bulk_g2s(dst + p.w_stage_bytes + T * 32, p.zeros + static_cast<size_t>(j) * N + 16 * tile0, sbytes, bar);
    };

    if (lane == 0) {
        for (int s = 0; s < p.nstage; ++s) mbar_init(my_bar + s * 8, 1);
        fence_barrier_init();
        fence_proxy_async();
        if (active) {
            const int pre = min(p.nstage, ng);
            for (int it = 0; it < pre; ++it) issue_chunk(it);
        }
    }
    __syncwarp();

    // Weights are in flight; let the next kernel begin its own prefetch, then wait until the
    // previous kernel has finished before x, y or the workspace are touched.
    pdl_launch_dependents();
    pdl_wait();

    // ---- stage x for this group range ---------------------------------------------------------
    const int kr = ng * SLIM_GROUP;                           // columns in this range
    {
        // raw copy + per-token max exponent; warp `warp` serves tokens warp, warp + 8
        for (int m = warp; m < M; m += kWarps) {
            const __half2* src = reinterpret_cast<const __half2*>(p.x + static_cast<size_t>(m) * p.K + g0 * SLIM_GROUP);
            uint32_t mx = 0;
            for (int i = lane; i < kr / 2; i += 32) {
                const uint32_t v = *reinterpret_cast<const uint32_t*>(src + i);
                *reinterpret_cast<uint32_t*>(smem + sm.xraw + (static_cast<size_t>(m) * kr + 2 * i) * 2) = v;
                mx = max(mx, max(v & 0x7fffu, (v >> 16) & 0x7fffu));
            }
            mx = __reduce_max_sync(0xffffffffu, mx);
            if (lane == 0) {
                const int e = max(static_cast<int>(mx >> 10), 1);   // biased exponent of the largest |x| (Inf/NaN: 31)
                reinterpret_cast<int*>(smem + sm.sexp)[m] = (mx == 0) ? 0 : 27 - e;  // max|x| * 2^S in [2^12, 2^13)
            }
        }
        if (tid == 0) {
            uint16_t* xslot = reinterpret_cast<uint16_t*>(smem + sm.xslot);
            int slot = 0;
            for (int i = 0; i < ng; ++i) { xslot[i] = static_cast<uint16_t>(slot); slot += slice_count(p.gt.bits[g0 + i]); }
            xslot[ng] = static_cast<uint16_t>(slot);
        }
        // zero the staging area (columns of absent tokens must read as 0) and the sums
        const int nslots_max = p.max_slots;
        uint4* z4 = reinterpret_cast<uint4*>(smem + sm.xs);
        for (int i = tid; i < nslots_max * 4 * NT * 16; i += kThreads) z4[i] = make_uint4(0, 0, 0, 0);
        float* sx = reinterpret_cast<float*>(smem + sm.sx);
        for (int i = tid; i < ng * 8 * NT; i += kThreads) sx[i] = 0.f;
    }
    __syncthreads();
    {
        const uint16_t* xslot = reinterpret_cast<const uint16_t*>(smem + sm.xslot);
        const int* sexp = reinterpret_cast<const int*>(smem + sm.sexp);
        const __half* xraw = reinterpret_cast<const __half*>(smem + sm.xraw);
        // one item = (token m, local group i, column kk): split x into 4 e5m2 pieces and scatter them
        const int items = M * kr;
        for (int it = tid; it < items; it += kThreads) {
            const int m = it / kr, rem = it - m * kr;
            const int i = rem >> 7, kk = rem & 127;
            const int b = p.gt.bits[g0 + i];
            const float xf = __half2float(xraw[static_cast<size_t>(m) * kr + rem]);
            const int S = sexp[m];
            const int nt = m >> 1, colbase = 4 * (m & 1);
            const int cc = kk >> 5, r32 = kk & 31;
            const int ns = slice_count(b);
            for (int s = 0; s < ns; ++s) {
                const int w = slice_w(b, s), lo = slice_lo(b, s);
                const int nf = 32 / w, per_byte = 8 / w;
                const int u = r32 / nf, f = r32 % nf;
                const int bt = f / per_byte, pp = f % per_byte;
                const int mi = u * (4 / w) + (pp >> 1), reg = pp & 1;
                const int e = S + lo - field_pos(w, pp);
                float v = xf * __int_as_float((127 + e) << 23);
                uint8_t* dst = smem + sm.xs + ((static_cast<size_t>(xslot[i] + s) * 4 + mi) * NT + nt) * 256 + reg * 4 + bt;
#pragma unroll
                for (int pc = 0; pc < 4; ++pc) {
                    const float piece = __uint_as_float(__float_as_uint(v) & 0xffe00000u);  // top 3 significant bits
                    v -= piece;                                                           // exact
                    const uint16_t hb = __half_as_ushort(__float2half_rz(piece));
                    dst[((colbase + pc) * 4 + cc) * 8] = static_cast<uint8_t>(hb >> 8);   // e5m2 = high byte of fp16
                }
            }
        }
        // per (token, group): 2^(S-9) * sum_k x, 8 lanes per sum, fixed order
        float* sx = reinterpret_cast<float*>(smem + sm.sx);
        const int sums = M * ng;
        for (int qb = warp * 4; qb < sums; qb += kThreads / 8) {     // warp-uniform trip count
            const int q = qb + (lane >> 3), l8 = lane & 7;
            const bool valid = q < sums;
            const int m = valid ? q / ng : 0, i = valid ? q - m * ng : 0;
            const __half* src = xraw + static_cast<size_t>(m) * kr + i * SLIM_GROUP + 16 * l8;
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < 16; ++k) acc += __half2float(src[k]);
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            acc += __shfl_xor_sync(0xffffffffu, acc, 2);
            acc += __shfl_xor_sync(0xffffffffu, acc, 4);
            if (valid && l8 == 0) sx[i * 8 * NT + (m >> 1) * 8 + 4 * (m & 1)] = acc * __int_as_float((127 + sexp[m] - 9) << 23);
        }
    }
    __syncthreads();

    // ---- main loop ------------------------------------------------------------------------------
    float acc[T][NT][4];
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[t][n][r] = 0.f;

    bool timed_out = false;
    int consumed = 0;   // chunks whose barrier phase has been observed
    if (active) {
        const uint16_t* xslot = reinterpret_cast<const uint16_t*>(smem + sm.xslot);
        constexpr bool kCacheB = (NT <= 2);
        for (int it = 0; it < ng; ++it) {
            const int st = it % p.nstage;
            if (!mbar_wait_bounded(my_bar + st * 8, (it / p.nstage) & 1)) { timed_out = true; break; }
            consumed = it + 1;
            const int b = p.gt.bits[g0 + it];
            const uint32_t stage = my_ring + st * p.stage_bytes;
            const uint32_t xs_slot0 = sbase + sm.xs + static_cast<uint32_t>(xslot[it]) * 4 * NT * 256;

            float d[T][NT][4];
#pragma unroll
            for (int t = 0; t < T; ++t)
#pragma unroll
                for (int n = 0; n < NT; ++n)
#pragma unroll
                    for (int r = 0; r < 4; ++r) d[t][n][r] = 0.f;

            // one slice of width W starting at unit `unit0`, activations in staging slot `xs_slot`
            auto run_slice = [&](auto wtag, int unit0, uint32_t xs_slot) {
                constexpr int W = decltype(wtag)::value;
                constexpr int MPU = 4 / W;                  // MMAs per unit
                uint2 bf[kCacheB ? 4 : 1][kCacheB ? NT : 1];
                if constexpr (kCacheB) {
#pragma unroll
                    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                        for (int n = 0; n < NT; ++n) bf[mi][n] = lds64(xs_slot + ((mi * NT + n) * 32 + lane) * 8);
                }
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    if (t < tw) {
#pragma unroll
                        for (int u = 0; u < W; ++u) {
                            const uint2 wd = lds64(stage + t * 256 * b + 256 * (unit0 + u) + 8 * lane);
                            const uint32_t sha = wd.x >> 4, shb = wd.y >> 4;
#pragma unroll
                            for (int ii = 0; ii < MPU; ++ii) {
                                const uint32_t a0 = field<W>(wd.x, sha, 2 * ii), a1 = field<W>(wd.y, shb, 2 * ii);
                                const uint32_t a2 = field<W>(wd.x, sha, 2 * ii + 1), a3 = field<W>(wd.y, shb, 2 * ii + 1);
                                const int mi = u * MPU + ii;
#pragma unroll
                                for (int n = 0; n < NT; ++n) {
                                    const uint2 bv = kCacheB ? bf[kCacheB ? mi : 0][kCacheB ? n : 0]
                                                             : lds64(xs_slot + ((mi * NT + n) * 32 + lane) * 8);
                                    mma_e4m3_e5m2(d[t][n], a0, a1, a2, a3, bv);
                                }
                            }
                        }
                    }
                }
            };
            switch (b) {
                case 1: run_slice(W1{}, 0, xs_slot0); break;
                case 2: run_slice(W2{}, 0, xs_slot0); break;
                case 3: run_slice(W2{}, 0, xs_slot0); run_slice(W1{}, 2, xs_slot0 + 4 * NT * 256); break;
                default: run_slice(W4{}, 0, xs_slot0); break;
            }

            // fold the group: acc += s * (D - z * sum_x)
            const uint32_t sxa = sbase + sm.sx + (it * 8 * NT + 2 * c) * 4;
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (t < tw) {
                    const uint32_t s2 = lds32(stage + p.w_stage_bytes + t * 32 + gq * 4);
                    const uint32_t z2 = lds32(stage + p.w_stage_bytes + T * 32 + t * 32 + gq * 4);
                    const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
                    const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&z2));
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        const uint2 sxr = lds64(sxa + n * 32);
                        const float sx0 = __uint_as_float(sxr.x), sx1 = __uint_as_float(sxr.y);
                        acc[t][n][0] = fmaf(sf.x, fmaf(-zf.x, sx0, d[t][n][0]), acc[t][n][0]);
                        acc[t][n][1] = fmaf(sf.x, fmaf(-zf.x, sx1, d[t][n][1]), acc[t][n][1]);
                        acc[t][n][2] = fmaf(sf.y, fmaf(-zf.y, sx0, d[t][n][2]), acc[t][n][2]);
                        acc[t][n][3] = fmaf(sf.y, fmaf(-zf.y, sx1, d[t][n][3]), acc[t][n][3]);
                    }
                }
            }
            // the stage is free again: refill it with the chunk nstage groups ahead
            __syncwarp();
            if (lane == 0 && it + p.nstage < ng) {
                fence_proxy_async();
                issue_chunk(it + p.nstage);
            }
        }
        if (timed_out) {
            // leave nothing in flight: every issued chunk either lands or its wait runs out as well
            if (lane == 0) {
                atomicOr(p.status, 1u);
                const int issued = min(ng, consumed + p.nstage);
                for (int it = consumed; it < issued; ++it)
                    (void)mbar_wait_bounded(my_bar + (it % p.nstage) * 8, (it / p.nstage) & 1);
            }
            __syncwarp();
        }
    }

    // ---- combine the piece columns of each token, scale back, write -------------------------------
    const int* sexp = reinterpret_cast<const int*>(smem + sm.sexp);
    const bool direct = (p.SK == 1);
#pragma unroll
    for (int t = 0; t < T; ++t) {
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            float va = acc[t][n][0] + acc[t][n][1];    // row 2gq,   columns 2c, 2c+1
            float vb = acc[t][n][2] + acc[t][n][3];    // row 2gq+1
            va += __shfl_xor_sync(0xffffffffu, va, 1);
            vb += __shfl_xor_sync(0xffffffffu, vb, 1);
            const int m = 2 * n + (c >> 1);
            if (active && t < tw && (c & 1) == 0 && m < M) {
                const float back = __int_as_float((127 + 9 - sexp[m]) << 23);
                va *= back;
                vb *= back;
                const int row = 16 * (tile0 + t) + 2 * gq;
                if (direct) {
                    *reinterpret_cast<__half2*>(p.y + static_cast<size_t>(m) * N + row) = __floats2half2_rn(va, vb);
                } else {
                    *reinterpret_cast<float2*>(p.partials + (static_cast<size_t>(ks) * M + m) * N + row) = make_float2(va, vb);
                }
            }
        }
    }
    if (direct) return;

    // ---- split-K: the last CTA of this row block adds the partials in split order ------------------
    __shared__ unsigned int s_ticket;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_ticket = atomicAdd(p.counters + rb, 1u);
    __syncthreads();
    if (s_ticket != static_cast<unsigned int>(p.SK - 1)) return;
    __threadfence();
    const int row0 = rb * kWarps * T * 16;
    const int nrows = min(kWarps * T * 16, N - row0);
    for (int i = tid; i < M * (nrows / 2); i += kThreads) {
        const int m = i / (nrows / 2), r2 = i - m * (nrows / 2);
        const size_t off = static_cast<size_t>(m) * N + row0 + 2 * r2;
        float2 sum = make_float2(0.f, 0.f);
        for (int s = 0; s < p.SK; ++s) {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(p.partials + static_cast<size_t>(s) * M * N + off));
            sum.x += v.x;
            sum.y += v.y;
        }
        *reinterpret_cast<__half2*>(p.y + off) = __floats2half2_rn(sum.x, sum.y);
    }
    if (tid == 0) p.counters[rb] = 0;   // leave the counter ready for the next call
}

// ------------------------------------------------------------------------------------------ host side
struct GemvPlan {
    int NT, T, SK, RB;
    int nstage, stage_bytes, w_stage_bytes;
    int max_groups, max_slots;
    uint32_t smem_bytes;
    uint16_t kbegin[kMaxSplit + 1];
    size_t counters_bytes, partial_bytes;
};

static int device_sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Deterministic launch plan for (M, N, K, bit map) on the current device.
static void plan_gemv(int M, int N, const GroupTable& gt, GemvPlan* pl) {
    const int G = gt.G;
    const int need_nt = (M + 1) / 2;
    pl->NT = need_nt <= 1 ? 1 : need_nt <= 2 ? 2 : need_nt <= 4 ? 4 : 8;
    pl->T = pl->NT <= 2 ? 2 : 1;
    const int rows_per_cta = kWarps * pl->T * 16;
    pl->RB = (N + rows_per_cta - 1) / rows_per_cta;
    int bmax = 1;
    for (int j = 0; j < G; ++j) bmax = bmax > gt.bits[j] ? bmax : gt.bits[j];
    pl->w_stage_bytes = pl->T * 256 * bmax;
    pl->stage_bytes = static_cast<int>(align_up(pl->w_stage_bytes + 2 * pl->T * 32, 128));

    const int sms = device_sm_count();
    int sk = sms / (pl->RB > 0 ? pl->RB : 1);
    if (sk < 1) sk = 1;
    if (sk > G) sk = G;
    if (sk > kMaxSplit) sk = kMaxSplit;
    const uint32_t smem_budget = 100 * 1024;   // two CTAs per SM: the next layer's CTA co-resides
    for (;; ++sk) {
        // boundaries at the group where the running bit count crosses i/sk of the total
        const int total = gt.prefix[G];
        pl->kbegin[0] = 0;
        int j = 0;
        for (int i = 1; i < sk; ++i) {
            const int target = (total * i + sk / 2) / sk;
            while (j < G && gt.prefix[j] < target) ++j;
            if (j <= pl->kbegin[i - 1]) j = pl->kbegin[i - 1] + 1;   // every split gets at least one group
            if (j > G - (sk - i)) j = G - (sk - i);
            pl->kbegin[i] = static_cast<uint16_t>(j);
        }
        pl->kbegin[sk] = static_cast<uint16_t>(G);
        int mg = 0, ms = 0;
        for (int i = 0; i < sk; ++i) {
            const int a = pl->kbegin[i], b = pl->kbegin[i + 1];
            int slots = 0;
            for (int q = a; q < b; ++q) slots += slice_count(gt.bits[q]);
            mg = mg > (b - a) ? mg : (b - a);
            ms = ms > slots ? ms : slots;
        }
        pl->max_groups = mg;
        pl->max_slots = ms;
        const SmemMap fixed = make_smem_map(pl->NT, M, 0, 0, mg, ms);
        const uint32_t ring_min = static_cast<uint32_t>(kWarps) * 2 * pl->stage_bytes;
        if (fixed.total + ring_min <= smem_budget || sk >= G || sk >= kMaxSplit) {
            const uint32_t avail = smem_budget > fixed.total ? smem_budget - fixed.total : 0;
            int ns = static_cast<int>(avail / (static_cast<uint32_t>(kWarps) * pl->stage_bytes));
            if (ns > kMaxStages) ns = kMaxStages;
            if (ns > mg) ns = mg;
            if (ns < 2) ns = mg < 2 ? 1 : 2;
            pl->nstage = ns;
            pl->smem_bytes = make_smem_map(pl->NT, M, ns, pl->stage_bytes, mg, ms).total;
            break;
        }
    }
    pl->SK = sk;
    pl->counters_bytes = align_up(4u * static_cast<uint32_t>(N / 128 + 1), 256);
    pl->partial_bytes = sk > 1 ? static_cast<size_t>(sk) * M * N * sizeof(float) : 0;
}

template <int NT, int T>
static cudaError_t launch_gemv(const GemvParams& prm, const GemvPlan& pl, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemv_kernel<NT, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(pl.RB), static_cast<unsigned>(pl.SK), 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_kernel<NT, T>, prm);
}

}  // namespace slim

extern "C" {

int slim_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes) {
    if (out_bytes == nullptr || M < 0) return SLIM_ERR_INVALID_ARG;
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    size_t bytes = slim::kWsHeader + slim::align_up(4u * static_cast<uint32_t>(N / 128 + 1), 256);
    if (M >= 1 && M <= SLIM_GEMV_MAX_M && N > 0 && K > 0) {
        slim::GemvPlan pl;
        slim::plan_gemv(M, N, gt, &pl);
        bytes += pl.partial_bytes;
    }
    *out_bytes = bytes;
    return SLIM_OK;
}

int slim_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (workspace == nullptr || workspace_bytes < slim::kWsHeader) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
    // control region = header + counters; zeroing the whole workspace is simplest and always safe
    SLIM_CUDA_TRY(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)));
    return SLIM_OK;
}

int slim_workspace_status(void* workspace, void* stream) {
    if (workspace == nullptr) return SLIM_ERR_WORKSPACE;
    unsigned int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SLIM_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, s));
    SLIM_CUDA_TRY(cudaStreamSynchronize(s));
    if (word != 0) {
        SLIM_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof word, s));
        SLIM_CUDA_TRY(cudaStreamSynchronize(s));
        return SLIM_ERR_TIMEOUT;
    }
    return SLIM_OK;
}

int slim_mpq_gemv(const void* x, const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros,
                  void* y, int M, int N, int K, int g, void* workspace, size_t workspace_bytes, void* stream) {
    if (M < 0 || M > SLIM_GEMV_MAX_M) return SLIM_ERR_INVALID_ARG;
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (M == 0 || N == 0) return SLIM_OK;
    if (y == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(y)) return SLIM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (K == 0) {  // empty reduction: y = 0
        SLIM_CUDA_TRY(cudaMemsetAsync(y, 0, static_cast<size_t>(M) * N * sizeof(__half), s));
        return SLIM_OK;
    }
    if (x == nullptr || packed == nullptr || scales == nullptr || zeros == nullptr) return SLIM_ERR_INVALID_ARG;
    if (!slim::aligned16(x) || !slim::aligned16(packed) || !slim::aligned16(scales) || !slim::aligned16(zeros))
        return SLIM_ERR_ALIGNMENT;

    slim::GemvPlan pl;
    slim::plan_gemv(M, N, gt, &pl);
    const size_t need = slim::kWsHeader + pl.counters_bytes + pl.partial_bytes;
    if (workspace == nullptr || workspace_bytes < need) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;

    slim::GemvParams prm;
    memset(&prm, 0, sizeof prm);
    prm.x = static_cast<const __half*>(x);
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.zeros = static_cast<const __half*>(zeros);
    prm.y = static_cast<__half*>(y);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    prm.status = reinterpret_cast<unsigned int*>(ws);
    prm.counters = reinterpret_cast<unsigned int*>(ws + slim::kWsHeader);
    prm.partials = reinterpret_cast<float*>(ws + slim::kWsHeader + pl.counters_bytes);
    prm.M = M; prm.N = N; prm.K = K;
    prm.SK = pl.SK;
    prm.nstage = pl.nstage;
    prm.stage_bytes = pl.stage_bytes;
    prm.w_stage_bytes = pl.w_stage_bytes;
    prm.max_groups = pl.max_groups;
    prm.max_slots = pl.max_slots;
    memcpy(prm.kbegin, pl.kbegin, sizeof prm.kbegin);
    prm.gt = gt;

    cudaError_t e;
    if (pl.NT == 1) e = slim::launch_gemv<1, 2>(prm, pl, s);
    else if (pl.NT == 2) e = slim::launch_gemv<2, 2>(prm, pl, s);
    else if (pl.NT == 4) e = slim::launch_gemv<4, 1>(prm, pl, s);
    else e = slim::launch_gemv<8, 1>(prm, pl, s);
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

}  // extern "C"
