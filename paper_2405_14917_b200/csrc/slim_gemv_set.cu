// slim_mpq_gemv_set: the decode path (1 <= M <= 16) over a set of independent layers, sm_100a.
//
// A decode-sized layer holds fewer bytes than HBM must keep in flight, so a launch per layer
// leaves the memory system idle while kernels start, stage x and reduce.  Here the whole set is
// one stream of work items for persistent CTAs:
//
//  * item = (layer, block of 128 or 256 rows = 8 tiles of 16 per consumer warp's share), the full K
//    of the layer.  The host deals the items to the CTAs, heaviest first, each to the CTA with the
//    least work so far, and writes every CTA's list into the plan.
//  * x is put into B-fragment order once per layer by a small kernel (one warp per token and
//    group; the routine slim_mpq_gemv uses) and kept in the workspace; every item re-reads its
//    fragments from L2.
//  * a producer warp walks the CTA's items group by group and brings, per group, the slices of the
//    8 tiles (one contiguous piece of the packed buffer), their scales and zeros, the group's
//    fragments and its (sum_k x, 2^(24-S)) into the next slot of a shared-memory ring with
//    cp.async.bulk; mbarriers hand the slots back and forth.  The ring never drains between items
//    or layers, so HBM always has the ring's worth of bytes in flight per CTA.
//  * consumer warp w owns tile w of the item: per group one pass of mma.sync m16n8k16 over raw
//    code fields (subnormal-mantissa operands, see slim_gemv_dev.cuh / slim_gemv.cu) and the fold
//    acc += s * (D * 2^(24-S) - z * sum_k x); after the last group it stores its 16 rows.  A warp
//    walks the whole K itself: no partial sums, no reduction between warps or CTAs.
//
// Every wait on an mbarrier is bounded and reports through the workspace status word.
#include "slim_gemv_dev.cuh"
#include "slim_gemv_i8.cuh"

#include <atomic>

#include <algorithm>
#include <cstring>
#include <exception>
#include <functional>
#include <queue>
#include <utility>
#include <vector>

namespace slim {

constexpr int kSetConsumers = 8;                       // consumer warps; each owns TPW (1 or 2) tiles of an item
constexpr int kSetProducers = 2;                       // producer warps: they take the groups in turn
constexpr int kSetThreads = 32 * (kSetConsumers + kSetProducers);
constexpr int kSetMaxSlots = 32;
constexpr int kSetCtasPerSm = 2;                       // resident CTAs per SM the plan aims at (one from 17 tokens on: registers)
constexpr int kSetMaxTokens = 64;                      // tokens of a layer in a set: up to eight MMA tiles of 8

// Layout of a ring slot (tpi = 16-row tiles of a work item, mp = 256-byte pieces per slice of the staged
// activations: 2 for single-token sets, else the 8 or 16 tokens of the set).  Everything but the packed slices has
// a fixed size, so the slices come last and every other offset is a compile-time constant of the kernel:
//   header (bit-width of the group) | scales | zeros | (sum_k x, scale) per token | activations of two slices | slices
constexpr int kSlotOffS = 16;
__host__ __device__ constexpr int slot_off_z(int tpi) { return kSlotOffS + 32 * tpi; }
__host__ __device__ constexpr int slot_off_e(int tpi) { return kSlotOffS + 64 * tpi; }
__host__ __device__ constexpr int slot_off_x(int tpi, int mp) { return slot_off_e(tpi) + (mp > 16 ? 8 * mp : 128); }
__host__ __device__ constexpr int slot_off_w(int tpi, int mp) { return slot_off_x(tpi, mp) + 2 * 256 * mp; }

// Device-side description of one layer (lives in the plan buffer).
struct SetLayer {
    const __half* x;
    const uint8_t* packed;
    const __half* scales;
    const __half* zeros;
    __half* y;
    size_t x_off;          // workspace offset of the layer's staged activations, group after group:
                           // (sum_k x, 2^(24-S)) float2[16], then the fragments [slice][8 mma][MP][4 lanes] x 8 B
    size_t part_off;       // workspace offset of the layer's fp32 partial outputs [split][M][N] (split > 1 only)
    int M, N, K, G;
    uint16_t count[4];     // groups of 1, 2, 3, 4 bits
    int task0;             // first (token, group) staging task of the layer
    int MP;                // 256-byte pieces per slice in the staged layout: 8 or 16 = tokens of the f16 fragments for the
                           // whole set (absent tokens are staged as zeros, so the kernel reads without a test); 2 if every
                           // layer of the set has one token: the 8-bit digit form (stage_group_i8)
    uint16_t prefix[SLIM_MAX_GROUPS + 1];
    uint16_t pre3[SLIM_MAX_GROUPS + 1];   // 3-bit groups (two slices) before group j
    uint8_t bits[SLIM_MAX_GROUPS];
    uint8_t order[SLIM_MAX_GROUPS];       // the order in which the groups are streamed: by bit-width, then by index
    uint8_t split;                        // parts the groups of a row block are cut into (1: whole K per item)
    uint8_t gshift;                       // 2^gshift K-tiles of 128 columns share a row of scales and zeros (g = 128 << gshift)
    uint16_t cnt0;                        // split > 1: the layer's first arrival counter (one per row block and consumer warp)
};
static_assert(sizeof(SetLayer) % 16 == 0, "descriptors are copied and read in 16-byte pieces");

// One work item as the CTAs read it: what a consumer warp needs is here, so that it never waits for
// the layer's descriptor.
struct SetItem {
    int layer, rb;         // layer of the set, row block inside the layer
    int N;
    int range;             // the item's groups: positions [range & 0xffff, range >> 16) of the layer's streaming order
    __half* y;             // the layer's y; for an item that covers part of the groups, the workspace offset of its fp32
                           // partial output [M][N] instead
    int M;
    int counts;            // the layer's groups of 1, 2 and 3 bits, 9 bits each (the rest has 4), i.e. where each width
                           // starts in the streaming order; bit 30: partial item
};
constexpr int kItemPartial = 1 << 30;
static_assert(sizeof(SetItem) == 32, "items are read as two 16-byte pieces");

// Plan buffer: int item_begin[grid + 1] (padded to kSetPlanHeader bytes), the descriptors, then the
// items in the order the CTAs take them: CTA c owns entries item_begin[c] .. item_begin[c + 1].
constexpr int kSetMaxGrid = 1023;
constexpr size_t kSetPlanHeader = 4096;

struct SetParams {
    const int* item_begin;
    const SetLayer* layers;
    const SetItem* items;
    uint8_t* ws;                           // workspace: status word, arrival counters, then the layers' fragments and sums
    int n_layers, n_slots, slot_bytes;
    int one;                               // 1: a multiplier the compiler cannot fold, for selects done as integer multiply-adds
};

// ------------------------------------------------------e offset kSetOffCounters) start every launch at zero.
constexpr uint32_t kSetOffCounters = 256;
__device__ __forceinline__ void stage_clear_counters(uint8_t* ws, int n_counters) {
    unsigned int* cnt = reinterpret_cast<unsigned int*>(ws + kSetOffCounters);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_counters; i += gridDim.x * blockDim.x) cnt[i] = 0u;
}

// Staging task `pi` of layer L (one warp): token pi / G, group pi % G.
__device__ __forceinline__ void stage_task(const SetLayer& L, uint8_t* ws, int pi, int lane) {
    const int m = pi / L.G, j = pi - m * L.G;        // m < MP
    uint8_t* grp = ws + L.x_off + staged_group_offset(j, L.pre3[j], L.MP);
    if (L.MP == 2) {                                     // single-token set: the 8-bit form, one task per group
        __shared__ int Xs[8][SLIM_GROUP];
        stage_group_i8(L.x + j * SLIM_GROUP, grp, L.bits[j], lane, Xs[threadIdx.x >> 5]);
        return;
    }
    float2* sxe = reinterpret_cast<float2*>(grp);
    if (m < L.M) {
        const float2 r = stage_group(L.x + static_cast<size_t>(m) * L.K + j * SLIM_GROUP, grp + staged_header_bytes(L.MP), L.bits[j], m, L.MP, lane);
        if (lane == 0) sxe[m] = r;
    } else {
        // a token the layer does not have: zero fragments in every slice of the group
        const int cc = lane & 3, mi = lane >> 2;
        for (int sl = 0; sl < slice_count(L.bits[j]); ++sl)
            *reinterpret_cast<uint2*>(grp + staged_header_bytes(L.MP) + (((static_cast<size_t>(sl) * 8 + mi) * L.MP + m) * 4 + cc) * 8) = make_uint2(0u, 0u);
    }
    if (m == 0)
        for (int t = lane; t < max(L.MP, 16); t += 32)
            if (t >= L.M) sxe[t] = make_float2(0.f, 1.f);                          // absent tokens read 0
}

// One warp per (layer, token, group): fragments and sums of the whole set, once.
__global__ void __launch_bounds__(256) gemv_set_stage_kernel(const SetLayer* __restrict__ layers, uint8_t* ws, int n_layers, int n_tasks,
                                                             int n_counters) {
    pdl_wait();                       // x may be the output of the kernel before; the workspace may still be read by it
    pdl_launch_dependents();
    stage_clear_counters(ws, n_counters);
    const int lane = threadIdx.x & 31;
    const int task = blockIdx.x * 8 + (threadIdx.x >> 5);
    // The layer of a task is the last one whose first task is not above it.  A search through the descriptors is a
    // chain of dependent loads from global memory (eight for the 224 layers of a 7B sweep, most of this kernel's time),
    // so a set of up to kStageTable layers first puts their first tasks into shared memory, all loads in flight at once.
    constexpr int kStageTable = 2048;
    __shared__ int first_task[kStageTable];
    const bool table = n_layers <= kStageTable;
    if (table) {
        for (int l = threadIdx.x; l < n_layers; l += blockDim.x) first_task[l] = layers[l].task0;
        __syncthreads();
    }
    if (task >= n_tasks) return;
    int lo = 0, hi = n_layers - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((table ? first_task[mid] : layers[mid].task0) <= task) lo = mid; else hi = mid - 1;
    }
    stage_task(layers[lo], ws, task - (table ? first_task[lo] : layers[lo].task0), lane);
}

// D = A * B with a zero accumulator input: starts an accumulation chain without clearing registers first.
__device__ __forceinline__ void mma_f16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y), "f"(0.f));
}


// A consumer warp that has stored its fp32 partial sums of a split row block (n_act tiles from tile0 on, M tokens)
// counts itself on the row block's counter of this warp.  The warp that counts last sees the other parts and adds all
// parts in part order, so the result does not depend on which part came last: y = fp16 of that sum.  Out of line: it
// runs once per item.
__device__ __noinline__ void finish_parts(const SetParams& p, int layer, int rb, int warp, int lane, int tile0, int n_act, int M, int N) {
    const SetLayer* L = p.layers + layer;
    __threadfence();                                    // this lane's partial sums before the count
    __syncwarp();
    unsigned int old = 0;
    if (lane == 0)
        old = atomicAdd(reinterpret_cast<unsigned int*>(p.ws + kSetOffCounters) + L->cnt0 + rb * kSetConsumers + warp, 1u);
    old = __shfl_sync(0xffffffffu, old, 0);
    const int S = L->split;
    if (static_cast<int>(old) + 1 != S) return;
    __threadfence();
    const float* part = reinterpret_cast<const float*>(p.ws + L->part_off);
    const size_t MN = static_cast<size_t>(M) * N;
    __half* y = L->y;
    // 16 * n_act rows x M tokens as pairs of rows: pair i of token m
    const int pairs = 8 * n_act;
    for (int i = lane; i < pairs * M; i += 32) {
        const int m = i / pairs, r = i - m * pairs;
        const size_t at = static_cast<size_t>(m) * N + 16 * tile0 + 2 * r;
        float2 sum = __ldcg(reinterpret_cast<const float2*>(part + at));
        for (int k = 1; k < S; ++k) {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(part + k * MN + at));
            sum.x += v.x;
            sum.y += v.y;
        }
        *reinterpret_cast<__half2*>(y + at) = __floats2half2_rn(sum.x, sum.y);
    }
}

// Slow path of a consumer's wait, kept out of line so that the loop around it stays small.
__device__ __noinline__ bool wait_full_slow(uint32_t bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, sb::wait(bar, parity, abort));
}

// Consumer warp of a single-token set: integer MMAs on byte-masked words (see stage_group_i8), then the fold
// acc += s (D 2^(-S-Pc) - z sum_x) per (row, group).  The loop is bound by instruction dispatch, above all by the
// half-rate integer/logic pipe, so everything that is not a mask runs on the multiply-add pipe: the two
// accumulation chains of a tile are added, and the tile of this lane pair is selected, by integer multiply-adds
// with 0 / 1 multipliers, and the integer sums become floats through the mantissa of 1.5 * 2^23.
template <int TPW>
__device__ __forceinline__ void consume_one(const SetParams& p, const uint32_t sbase, const uint32_t ring, volatile int* abort,
                                            const int i0, const int i1, const int warp, const int lane) {
    auto full = [&](int s) { return sbase + 8u * s; };
    auto empty = [&](int s) { return sbase + 8u * (kSetMaxSlots + s); };
    constexpr int TPI = kSetConsumers * TPW, CHI = 2;
    constexpr uint32_t kOffZ = slot_off_z(TPI), kOffE = slot_off_e(TPI), kOffX = slot_off_x(TPI, 2), kOffW = slot_off_w(TPI, 2);
    static_assert(TPW <= 2, "one lane pair per tile");
    const int gq = lane >> 2, c = lane & 3;
    const int tsel = TPW == 2 ? (c >> 1) : 0;
    const int m0 = tsel ? 0 : p.one, m1 = tsel ? p.one : 0;
    // lanes with even c hold the sums of the two high digits, odd c of the two low ones
    const float ma = (c & 1) ? 256.f : 16777216.f, mb = (c & 1) ? 1.f : 65536.f;
    constexpr int kMagicBits = 0x4B400000;                 // 1.5 * 2^23: adding an integer |v| < 2^22 to these bits gives the float 12582912 + v
    constexpr float kMagic = 12582912.f;
    const uint32_t lane0 = lane == 0 ? 1u : 0u;
    const uint32_t slot_bytes = static_cast<uint32_t>(p.slot_bytes);
    const int n_slots = p.n_slots;
    const uint32_t sz_lane = static_cast<uint32_t>((TPW * warp + tsel) * 32 + gq * 4);
    const uint32_t x_lane = kOffX + ((gq & 3) * 4 + c) * 8;
    const uint32_t w_lane = kOffW + 8u * lane;
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    const int4* items4 = reinterpret_cast<const int4*>(p.items);
    int4 it_a = items4[2 * i0], it_b = items4[2 * i0 + 1];       // (layer, rb, N, G), (y, M, counts)
    for (int i = i0; i < i1 && ok; ++i) {
        const int layer = it_a.x, rb = it_a.y, N = it_a.z, p0 = it_a.w & 0xffff, p1 = it_a.w >> 16, counts = it_b.w;
        const int G = p1 - p0;                                   // groups of this item
        const unsigned long long yword = (static_cast<unsigned long long>(static_cast<uint32_t>(it_b.y)) << 32) | static_cast<uint32_t>(it_b.x);
        if (i + 1 < i1) {                                        // the next item arrives during this one's groups
            it_a = items4[2 * i + 2];
            it_b = items4[2 * i + 3];
        }
        const int tile0 = TPI * rb + TPW * warp;
        const int n_act = min(TPW, (N >> 4) - tile0);
        if (n_act <= 0) {
            // a warp whose tiles lie past the end of the layer only hands the slots back
            for (int j = 0; j < G; ++j) {
                if (!__all_sync(0xffffffffu, sb::try_wait(full(s), ph)) && !wait_full_slow(full(s), ph, abort)) { ok = false; break; }
                __syncwarp();
                sb::arrive_if(empty(s), lane0);
                if (++s == n_slots) { s = 0; ph ^= 1u; }
            }
            continue;
        }
        float acc0 = 0.f, acc2 = 0.f;

        // The groups of an item arrive sorted by bit-width (the counts come with the item), so each width has a loop
        // of its own and no group has to say what it is.  `n` groups of B bits: false if a wait gave up.
        auto run_groups = [&](auto btag, int n) -> bool {
            constexpr int B = decltype(btag)::value;
            for (int k = 0; k < n; ++k) {
                if (!__all_sync(0xffffffffu, sb::try_wait(full(s), ph)) && !wait_full_slow(full(s), ph, abort)) return false;
                const uint32_t slot = ring + static_cast<uint32_t>(s) * slot_bytes;
                // tile t of the warp: its slices follow each other.  For a tile past the end of the layer the slot holds
                // stale bytes: its sums are computed and never stored.
                const uint32_t item0 = slot + w_lane + static_cast<uint32_t>(TPW * warp) * (256u * B);
                const uint32_t xs_lane = slot + x_lane;
                int di[TPW][CHI][4];
                // one slice of width WD starting at unit `unit0`, digits at `xs`
                auto run_pass = [&](auto wtag, auto first_tag, int unit0, uint32_t xs) {
                    constexpr int WD = decltype(wtag)::value;
                    constexpr bool FIRST = decltype(first_tag)::value != 0;
                    constexpr uint32_t kByteMask = 0x01010101u * ((1u << WD) - 1u);
                    constexpr int NW = WD;                  // 8-byte pieces (two rows' words) per lane that the MMAs of the slice draw on
                    uint2 wd[TPW][NW];
#pragma unroll
                    for (int t = 0; t < TPW; ++t) {
                        const uint32_t item = item0 + t * (256u * B) + 256u * unit0;
#pragma unroll
                        for (int u = 0; u < NW; ++u) wd[t][u] = lds64(item + 256u * u);
                    }
#pragma unroll
                    for (int mi = 0; mi < 4; ++mi) {
                        const uint2 bv = lds64(xs + mi * 128);
                        // registers (a0, a1) meet the MMA's k < 16, (a2, a3) its k >= 16: for a 1-bit slice field positions mi and
                        // mi + 4 of the same word, else position mi (mi & 1 for 4 bits) of two consecutive words.  The top position of
                        // a byte takes the word unmasked (its digits are made for that).
                        const int w_lo = WD == 4 ? 2 * (mi >> 1) : 0, w_hi = WD == 1 ? 0 : w_lo + 1;
                        const int pos_lo = i8_pos(WD, mi, 0), pos_hi = i8_pos(WD, mi, 1);
                        const uint32_t m_lo = kByteMask << (WD * pos_lo), m_hi = kByteMask << (WD * pos_hi);
                        const bool top_lo = WD * (pos_lo + 1) == 8, top_hi = WD * (pos_hi + 1) == 8;
#pragma unroll
                        for (int t = 0; t < TPW; ++t) {
                            const uint32_t a0 = top_lo ? wd[t][w_lo].x : wd[t][w_lo].x & m_lo, a1 = top_lo ? wd[t][w_lo].y : wd[t][w_lo].y & m_lo;
                            const uint32_t a2 = top_hi ? wd[t][w_hi].x : wd[t][w_hi].x & m_hi, a3 = top_hi ? wd[t][w_hi].y : wd[t][w_hi].y & m_hi;
                            if (FIRST && mi < CHI) mma_i8_first(di[t][mi & (CHI - 1)], a0, a1, a2, a3, bv);
                            else mma_i8(di[t][mi & (CHI - 1)], a0, a1, a2, a3, bv);
                        }
                    }
                };
                if (B == 1) run_pass(W1{}, WidthTag<1>{}, 0, xs_lane);
                if (B == 2) run_pass(W2{}, WidthTag<1>{}, 0, xs_lane);
                if (B == 3) { run_pass(W2{}, WidthTag<1>{}, 0, xs_lane); run_pass(W1{}, WidthTag<0>{}, 2, xs_lane + 512); }
                if (B == 4) run_pass(W4{}, WidthTag<1>{}, 0, xs_lane);
                // fold.  Columns (0, 1) hold the sums of the two high digits, (2, 3) of the two low ones, (4..7) repeat
                // them.  Every lane holds the sums of all the warp's tiles; the lane pair c >> 1 folds tile c >> 1.
                const uint2 tkw = lds64(slot + kOffE);
                const uint32_t s2 = lds32(slot + kSlotOffS + sz_lane);
                const uint32_t z2 = lds32(slot + kOffZ + sz_lane);
                const float sum_x = __uint_as_float(tkw.x), e = __uint_as_float(tkw.y);
                const float ka = ma * e, kb = mb * e;
                float f[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    int v = kMagicBits;
#pragma unroll
                    for (int ch = 0; ch < CHI; ++ch) v += di[0][ch][r] * m0 + di[TPW - 1][ch][r] * m1;
                    f[r] = __int_as_float(v) - kMagic;                        // exact
                }
                const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
                const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&z2));
                float r0 = fmaf(f[0], ka, f[1] * kb);
                float r1 = fmaf(f[2], ka, f[3] * kb);
                r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
                r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
                acc0 = fmaf(sf.x, fmaf(-zf.x, sum_x, r0), acc0);
                acc2 = fmaf(sf.y, fmaf(-zf.y, sum_x, r1), acc2);
                __syncwarp();
                sb::arrive_if(empty(s), lane0);
                if (++s == n_slots) { s = 0; ph ^= 1u; }
            }
            return true;
        };
        // the widths start at positions 0, e1, e2, e3 of the layer's streaming order; the item covers [p0, p1)
        const int e1 = counts & 511, e2 = e1 + ((counts >> 9) & 511), e3 = e2 + ((counts >> 18) & 511);
        auto part = [&](int a, int b) { return max(min(p1, b) - max(p0, a), 0); };
        ok = run_groups(WidthTag<1>{}, part(0, e1)) && run_groups(WidthTag<2>{}, part(e1, e2)) &&
             run_groups(WidthTag<3>{}, part(e2, e3)) && run_groups(WidthTag<4>{}, part(e3, 65535));
        if (ok) {
#pragma unroll
            for (int t = 0; t < TPW; ++t) {
                if (t >= n_act) break;
                const int row = 16 * (tile0 + t) + 2 * gq;
                if (c == 2 * t) {
                    if (counts & kItemPartial) *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.ws + yword) + row) = make_float2(acc0, acc2);
                    else *reinterpret_cast<__half2*>(reinterpret_cast<__half*>(yword) + row) = __floats2half2_rn(acc0, acc2);
                }
            }
            if (counts & kItemPartial) finish_parts(p, layer, rb, warp, lane, tile0, n_act, 1, N);
        }
    }
}


// Consumer warp of a set with more than one token somewhere: f16 MMAs on raw code fields (one AND per operand
// register of two codes, see slim_gemv_dev.cuh), NT tiles of 8 tokens, then the fold
// acc += s (D 2^(24-S) - z sum_x) per (row, token, group).  Same loop structure as consume_one.
template <int NT, int TPW>
__device__ __forceinline__ void consume_f16(const SetParams& p, const uint32_t sbase, const uint32_t ring, volatile int* abort,
                                            const int i0, const int i1, const int warp, const int lane) {
    auto full = [&](int s) { return sbase + 8u * s; };
    auto empty = [&](int s) { return sbase + 8u * (kSetMaxSlots + s); };
    constexpr int TPI = kSetConsumers * TPW, MPK = 8 * NT;
    // interleaved accumulation chains per (tile, token tile): with four (tile, token tile) pairs the MMAs of one pair are far
    // enough apart without a second chain
    constexpr int CH = NT * TPW >= 4 ? 1 : (NT == 1 ? (TPW == 1 ? 4 : 2) : 2);
    constexpr uint32_t kOffZ = slot_off_z(TPI), kOffE = slot_off_e(TPI), kOffX = slot_off_x(TPI, MPK), kOffW = slot_off_w(TPI, MPK);
    const int gq = lane >> 2, c = lane & 3;
    const uint32_t lane0 = lane == 0 ? 1u : 0u;
    const uint32_t slot_bytes = static_cast<uint32_t>(p.slot_bytes);
    const int n_slots = p.n_slots;
    const uint32_t sz_lane = static_cast<uint32_t>(TPW * warp * 32 + gq * 4);
    const uint32_t x_lane = kOffX + (gq * 4 + c) * 8;             // fragment of token gq of the first token tile
    const uint32_t e_lane = kOffE + 16u * c;                      // (sum_x, scale) of tokens 2c, 2c + 1
    const uint32_t w_lane = kOffW + 8u * lane;
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    const int4* items4 = reinterpret_cast<const int4*>(p.items);
    int4 it_a = items4[2 * i0], it_b = items4[2 * i0 + 1];       // (layer, rb, N, range), (y, M, counts)
    for (int i = i0; i < i1 && ok; ++i) {
        const int layer = it_a.x, rb = it_a.y, N = it_a.z, p0 = it_a.w & 0xffff, p1 = it_a.w >> 16, M = it_b.z, counts = it_b.w;
        const unsigned long long yword = (static_cast<unsigned long long>(static_cast<uint32_t>(it_b.y)) << 32) | static_cast<uint32_t>(it_b.x);
        if (i + 1 < i1) {                                        // the next item arrives during this one's groups
            it_a = items4[2 * i + 2];
            it_b = items4[2 * i + 3];
        }
        const int tile0 = TPI * rb + TPW * warp;                 // this warp's first tile of the layer
        const int n_act = min(TPW, (N >> 4) - tile0);            // its tiles that exist (<= 0: none)
        if (n_act <= 0) {
            for (int j = p0; j < p1; ++j) {                      // only hands the slots back
                if (!__all_sync(0xffffffffu, sb::try_wait(full(s), ph)) && !wait_full_slow(full(s), ph, abort)) { ok = false; break; }
                __syncwarp();
                sb::arrive_if(empty(s), lane0);
                if (++s == n_slots) { s = 0; ph ^= 1u; }
            }
            continue;
        }
        float acc[TPW][NT][4];
#pragma unroll
        for (int t = 0; t < TPW; ++t)
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int r = 0; r < 4; ++r) acc[t][n][r] = 0.f;

        auto run_groups = [&](auto btag, int n_groups) -> bool {
            constexpr int B = decltype(btag)::value;
            for (int k = 0; k < n_groups; ++k) {
                if (!__all_sync(0xffffffffu, sb::try_wait(full(s), ph)) && !wait_full_slow(full(s), ph, abort)) return false;
                const uint32_t slot = ring + static_cast<uint32_t>(s) * slot_bytes;
                // tile t of the warp: its slices follow each other.  For a tile past the end of the layer the slot holds
                // stale bytes: its accumulators are computed and never stored.
                const uint32_t item0 = slot + w_lane + static_cast<uint32_t>(TPW * warp) * (256u * B);
                float d[TPW][CH][NT][4];      // every chain is started by an MMA with a zero accumulator
                // one slice of width WD starting at unit `unit0`, activations in fragment slot `xs`
                auto run_slice = [&](auto wtag, auto first_tag, int unit0, uint32_t xs) {
                    constexpr int WD = decltype(wtag)::value;
                    constexpr int MPU = 8 / WD;                 // MMAs per unit
                    constexpr bool FIRST = decltype(first_tag)::value != 0;   // the group's first slice
#pragma unroll
                    for (int u = 0; u < WD; ++u) {
                        uint2 wd[TPW];
                        uint32_t shx[TPW], shy[TPW];
#pragma unroll
                        for (int t = 0; t < TPW; ++t) {
                            wd[t] = lds64(item0 + t * (256u * B) + 256u * (unit0 + u));
                            shx[t] = wd[t].x >> pair_shift(WD);
                            shy[t] = wd[t].y >> pair_shift(WD);
                        }
#pragma unroll
                        for (int ii = 0; ii < MPU; ++ii) {
                            const int mi = u * MPU + ii;
#pragma unroll
                            for (int n = 0; n < NT; ++n) {
                                // fragment of token 8n + gq (tokens the layer lacks are staged as zeros)
                                const uint2 bv = lds64(xs + ((mi * MPK + 8 * n) * 4) * 8);
#pragma unroll
                                for (int t = 0; t < TPW; ++t) {
                                    const uint32_t a0 = pair<WD>(wd[t].x, shx[t], 2 * ii), a1 = pair<WD>(wd[t].y, shy[t], 2 * ii);
                                    const uint32_t a2 = pair<WD>(wd[t].x, shx[t], 2 * ii + 1), a3 = pair<WD>(wd[t].y, shy[t], 2 * ii + 1);
                                    if (FIRST && mi < CH) mma_f16_first(d[t][mi & (CH - 1)][n], a0, a1, a2, a3, bv);
                                    else mma_f16(d[t][mi & (CH - 1)][n], a0, a1, a2, a3, bv);
                                }
                            }
                        }
                    }
                };
                const uint32_t xs0 = slot + x_lane;
                if (B == 1) run_slice(W1{}, WidthTag<1>{}, 0, xs0);
                if (B == 2) run_slice(W2{}, WidthTag<1>{}, 0, xs0);
                if (B == 3) { run_slice(W2{}, WidthTag<1>{}, 0, xs0); run_slice(W1{}, WidthTag<0>{}, 2, xs0 + 8 * MPK * 32); }
                if (B == 4) run_slice(W4{}, WidthTag<1>{}, 0, xs0);
                // fold the group: rows 2gq, 2gq+1, tokens 8n+2c, 8n+2c+1
#pragma unroll
                for (int t = 0; t < TPW; ++t) {
                    const uint32_t s2 = lds32(slot + kSlotOffS + sz_lane + t * 32);
                    const uint32_t z2 = lds32(slot + kOffZ + sz_lane + t * 32);
                    const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
                    const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&z2));
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        const uint4 tkw = lds128(slot + e_lane + 64u * n);       // (sx0, e0, sx1, e1)
                        const float sx0 = __uint_as_float(tkw.x), e0 = __uint_as_float(tkw.y);
                        const float sx1 = __uint_as_float(tkw.z), e1 = __uint_as_float(tkw.w);
                        float dd[4];
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            dd[r] = CH == 1 ? d[t][0][n][r] : d[t][0][n][r] + d[t][CH > 1 ? 1 : 0][n][r];
                            if (CH == 4) dd[r] += d[t][2 % CH][n][r] + d[t][3 % CH][n][r];
                        }
                        acc[t][n][0] = fmaf(sf.x, fmaf(-zf.x, sx0, dd[0] * e0), acc[t][n][0]);
                        acc[t][n][1] = fmaf(sf.x, fmaf(-zf.x, sx1, dd[1] * e1), acc[t][n][1]);
                        acc[t][n][2] = fmaf(sf.y, fmaf(-zf.y, sx0, dd[2] * e0), acc[t][n][2]);
                        acc[t][n][3] = fmaf(sf.y, fmaf(-zf.y, sx1, dd[3] * e1), acc[t][n][3]);
                    }
                }
                __syncwarp();
                sb::arrive_if(empty(s), lane0);
                if (++s == n_slots) { s = 0; ph ^= 1u; }
            }
            return true;
        };
        // the widths start at positions 0, e1, e2, e3 of the layer's streaming order; the item covers [p0, p1)
        const int e1 = counts & 511, e2 = e1 + ((counts >> 9) & 511), e3 = e2 + ((counts >> 18) & 511);
        auto part = [&](int a, int b) { return max(min(p1, b) - max(p0, a), 0); };
        ok = run_groups(WidthTag<1>{}, part(0, e1)) && run_groups(WidthTag<2>{}, part(e1, e2)) &&
             run_groups(WidthTag<3>{}, part(e2, e3)) && run_groups(WidthTag<4>{}, part(e3, 65535));
        // ---- this warp's rows of the item: rows 2gq, 2gq+1 of tokens 8n+2c, 8n+2c+1 of every tile
        if (ok) {
            const bool partial = (counts & kItemPartial) != 0;
#pragma unroll
            for (int t = 0; t < TPW; ++t) {
                if (t >= n_act) break;
                const int row = 16 * (tile0 + t) + 2 * gq;
#pragma unroll
                for (int n = 0; n < NT; ++n) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {                    // tokens 8n + 2c and 8n + 2c + 1
                        const int m = 8 * n + 2 * c + q;
                        if (m >= M) continue;
                        const size_t at = static_cast<size_t>(m) * N + row;
                        if (partial) *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.ws + yword) + at) = make_float2(acc[t][n][q], acc[t][n][2 + q]);
                        else *reinterpret_cast<__half2*>(reinterpret_cast<__half*>(yword) + at) = __floats2half2_rn(acc[t][n][q], acc[t][n][2 + q]);
                    }
                }
            }
            if (partial) finish_parts(p, layer, rb, warp, lane, tile0, n_act, M, N);
        }
    }
}

// ------------------------------------------------------------------------------------------ the persistent kernel
constexpr uint32_t kSetOffAbort = 16 * kSetMaxSlots;          // after the full and empty barriers
constexpr uint32_t kSetOffDesc = 1024;                        // the producer's copy of its layer's descriptor
constexpr uint32_t kSetOffRing = (kSetOffDesc + kSetProducers * sizeof(SetLayer) + 127) / 128 * 128;

// NT: 8-token MMA tiles, 1 (every M <= 8) or 2.  ONE: every layer has a single token; then only
// column 0 of the MMA results is ever used, so every lane feeds token 0's fragment and folds token 0.
// TPW: 16-row tiles per consumer warp (an item is 8 * TPW tiles; always 2 today); two tiles share the fragment
// loads and the per-group bookkeeping.
template <int NT, bool ONE, int TPW>
__global__ void __launch_bounds__(kSetThreads, NT >= 4 ? 1 : kSetCtasPerSm) gemv_set_kernel(const __grid_constant__ SetParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto full = [&](int s) { return sbase + 8u * s; };
    auto empty = [&](int s) { return sbase + 8u * (kSetMaxSlots + s); };
    volatile int* abort = reinterpret_cast<volatile int*>(smem + kSetOffAbort);
    const uint32_t ring = sbase + kSetOffRing;
    constexpr int TPI = kSetConsumers * TPW;                  // tiles per item
    constexpr uint32_t kOffZ = slot_off_z(TPI), kOffE = slot_off_e(TPI), kOffX = slot_off_x(TPI, ONE ? 2 : 8 * NT);
    constexpr uint32_t kOffW = slot_off_w(TPI, ONE ? 2 : 8 * NT);

    if (tid == 0) {
        for (int s = 0; s < p.n_slots; ++s) { sb::init(full(s), 1); sb::init(empty(s), kSetConsumers); }
        *abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Launched with programmatic stream serialization: everything above ran while the kernel before (the staging
    // kernel of this set) was still finishing; nothing of the plan or the workspace is read before it has completed.
    // The kernel after this one may be set up early in turn (ours wait in the same way before they touch memory).
    pdl_wait();
    pdl_launch_dependents();

    const int i0 = p.item_begin[blockIdx.x], i1 = p.item_begin[blockIdx.x + 1];
    if (i0 < i1) {
        if (warp >= kSetConsumers) {
            // -------------------------------------------------------------- producers
            // producer warp w takes the groups whose running number is w modulo the number of producers
            const int pw = warp - kSetConsumers;
            uint8_t* desc = smem + kSetOffDesc + pw * sizeof(SetLayer);
            const SetLayer* D = reinterpret_cast<const SetLayer*>(desc);
            int have = -1;                                // layer whose descriptor is in shared memory
            // ring position of the next group this warp fills: it advances by the number of producers
            int s = pw;
            uint32_t ph = 0;
            uint32_t cnt = 0;                             // running number of the group in this CTA's range
            bool ok = true;
            int l = p.items[i0].layer, rb = p.items[i0].rb, range = p.items[i0].range;
            for (int i = i0; i < i1 && ok; ++i) {
                // the next item's place is fetched while this one's groups are issued
                const int l_next = i + 1 < i1 ? p.items[i + 1].layer : 0, rb_next = i + 1 < i1 ? p.items[i + 1].rb : 0;
                const int range_next = i + 1 < i1 ? p.items[i + 1].range : 0;
                if (have != l) {
                    const uint4* src = reinterpret_cast<const uint4*>(p.layers + l);
                    uint4* dst = reinterpret_cast<uint4*>(desc);
                    for (int q = lane; q < static_cast<int>(sizeof(SetLayer) / 16); q += 32) dst[q] = src[q];
                    __syncwarp();
                    have = l;
                }
                const int N = D->N, MP = D->MP;
                const int p0 = range & 0xffff, p1 = range >> 16;        // the item's positions in the streaming order
                const int tiles_here = min(TPI, (N >> 4) - TPI * rb);
                // lane 0 brings the slices, lanes 1 and 2 scales and zeros, lane 3 the staged activations
                const uint8_t* base = lane == 0 ? D->packed
                                    : lane == 1 ? reinterpret_cast<const uint8_t*>(D->scales + 16 * TPI * rb)
                                    : lane == 2 ? reinterpret_cast<const uint8_t*>(D->zeros + 16 * TPI * rb)
                                                : p.ws + D->x_off;
                const uint32_t dst_off = lane == 0 ? kOffW : lane == 1 ? kSlotOffS : lane == 2 ? kOffZ : kOffE;
                const uint32_t szb = static_cast<uint32_t>(tiles_here) * 32u;
                int jj = p0 + static_cast<int>((static_cast<uint32_t>(pw) + kSetProducers - cnt % kSetProducers) % kSetProducers);
                cnt += static_cast<uint32_t>(p1 - p0);
                for (; jj < p1; jj += kSetProducers) {
                    // the lanes go on, or give up, together
                    if (!__all_sync(0xffffffffu, sb::wait(empty(s), ph ^ 1u, abort))) { ok = false; break; }
                    const int j = D->order[jj];            // the groups are streamed sorted by bit-width
                    const uint32_t b = D->bits[j];
                    const uint32_t wbytes = static_cast<uint32_t>(tiles_here) * 256u * b;
                    const uint32_t xbytes = static_cast<uint32_t>(staged_header_bytes(MP)) + static_cast<uint32_t>(slice_count(b)) * 256u * MP;
                    const uint32_t slot = ring + static_cast<uint32_t>(s) * p.slot_bytes;
                    if (lane == 0) {
                        asm volatile("st.shared.u32 [%0], %1;" ::"r"(slot), "r"(b) : "memory");
                        sb::expect_tx(full(s), wbytes + 2 * szb + xbytes);
                    }
                    const size_t off = lane == 0 ? 16ull * N * D->prefix[j] + static_cast<size_t>(TPI * rb) * 256 * b
                                     : lane == 3 ? staged_group_offset(j, D->pre3[j], MP)
                                                 : 2ull * static_cast<size_t>(j >> D->gshift) * N;
                    const uint32_t bytes = lane == 0 ? wbytes : lane == 3 ? xbytes : szb;
                    __syncwarp();
                    if (lane < 4) sb::bulk_g2s(slot + dst_off, base + off, bytes, full(s));
                    s += kSetProducers;
                    if (s >= p.n_slots) { s -= p.n_slots; ph ^= 1u; }
                }
                l = l_next;
                rb = rb_next;
                range = range_next;
            }
            if (!ok && lane == 0) {
                // leave no copy in flight: give what was issued a millisecond to land
                const unsigned long long t0 = sb::timer_ns();
                while (sb::timer_ns() - t0 < 1000000ull) { }
            }
        } else {
            // -------------------------------------------------------------- consumer: tile `warp` of every item
            if constexpr (ONE) consume_one<TPW>(p, sbase, ring, abort, i0, i1, warp, lane);
            else consume_f16<NT, TPW>(p, sbase, ring, abort, i0, i1, warp, lane);
        }
    }
    __syncthreads();
    if (tid == 0 && *abort != 0) atomicOr(reinterpret_cast<unsigned int*>(p.ws), 1u);
}

// ------------------------------------------------------------------------------------------ one-layer sets planned on the device
// Plan and staging of a one-layer set in one kernel: the descriptor comes by value, every warp stages one (token, group)
// of x, and block 0 also writes the plan: the items are (row block, part) pairs dealt to the CTAs in turn.  No host
// memory is read after the call has returned, so the call can be captured in a CUDA graph (slim_mpq_gemv sends its
// large layers this way).
__global__ void __launch_bounds__(256) set_single_stage_kernel(const __grid_constant__ SetLayer d, uint8_t* plan, uint8_t* ws, int grid,
                                                               int n_rb, int sp, int n_tasks, int n_counters) {
    pdl_wait();                       // x may be the output of the kernel before; the workspace may still be read by it
    pdl_launch_dependents();
    stage_clear_counters(ws, n_counters);
    if (blockIdx.x == 0) {
        int* item_begin = reinterpret_cast<int*>(plan);
        SetLayer* dl = reinterpret_cast<SetLayer*>(plan + kSetPlanHeader);
        SetItem* items = reinterpret_cast<SetItem*>(dl + 1);
        const int n = n_rb * sp, q = n / grid, r = n % grid;
        for (int c = threadIdx.x; c <= grid; c += blockDim.x) item_begin[c] = c * q + min(c, r);
        const uint4* src = reinterpret_cast<const uint4*>(&d);
        for (int i = threadIdx.x; i < static_cast<int>(sizeof(SetLayer) / 16); i += blockDim.x) reinterpret_cast<uint4*>(dl)[i] = src[i];
        for (int k = threadIdx.x; k < n; k += blockDim.x) {
            const int c = k % grid, t = k / grid;                // CTA c takes items c, c + grid, ...
            const int rb = k / sp, part = k - rb * sp;
            const int p0 = d.G * part / sp, p1 = d.G * (part + 1) / sp;
            SetItem it;
            it.layer = 0; it.rb = rb; it.N = d.N; it.range = p0 | (p1 << 16); it.M = d.M;
            it.counts = d.count[0] | (d.count[1] << 9) | (d.count[2] << 18) | (sp > 1 ? kItemPartial : 0);
            it.y = sp > 1 ? reinterpret_cast<__half*>(d.part_off + static_cast<size_t>(part) * d.M * d.N * sizeof(float)) : d.y;
            items[c * q + min(c, r) + t] = it;
        }
    }
    const int task = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (task < n_tasks) stage_task(d, ws, task, threadIdx.x & 31);
}

// ------------------------------------------------------------------------------------------ self-test of the bounded wait
// One warp waits, with the bounded wait of the persistent kernel, on an mbarrier that nobody arrives on.  When the
// limit has passed it raises the abort flag and the kernel reports through the workspace status word exactly as
// gemv_set_kernel does, then returns: the path a real time-out takes, without starving a real kernel.
__global__ void __launch_bounds__(32) wait_selftest_kernel(uint8_t* ws, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        sb::init(b, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = __all_sync(0xffffffffu, sb::wait_limit(b, 0, &abort_flag, limit_ns));
    __syncwarp();
    if (threadIdx.x == 0 && (!ok || abort_flag != 0)) atomicOr(reinterpret_cast<unsigned int*>(ws), 1u);
}

// ------------------------------------------------------------------------------------------ host side
// What the whole set fixes: token tiles, slot geometry, ring depth, grid, sizes.
struct SetGeometry {
    int nt, bmax, mmax, tpw, mpad;     // tpw: tiles per consumer warp; mpad: tokens in the staged layout
    int slot_bytes;
    int n_slots, grid, ctas_per_sm;
    int split;                         // parts the groups of every row block are cut into (fewer for layers with few groups)
    size_t smem_bytes;
    long long n_items, n_tasks;
    int n_counters;                    // arrival counters of the split row blocks: one per (row block, consumer warp)
    size_t cnt_bytes;                  // their room in the workspace, right after the 256-byte header
    size_t ws_bytes;
};
constexpr int kSetMaxSplit = 8;
constexpr int kSetMinGroupsPerPart = 4;
// Parts of a layer with G groups when the set asks for `split`.
static int layer_split(int split, int G) {
    const int cap = G / kSetMinGroupsPerPart > 1 ? G / kSetMinGroupsPerPart : 1;
    return split < cap ? split : cap;
}

static size_t align_to(size_t v, size_t a) { return (v + a - 1) / a * a; }
// Workspace of one layer: per group the sums and the fragments of its slices.
static size_t layer_ws_bytes(int M, const GroupTable& gt) {
    int slots = gt.G;
    for (int j = 0; j < gt.G; ++j) slots += gt.bits[j] == 3 ? 1 : 0;
    return align_to(static_cast<size_t>(gt.G) * staged_header_bytes(M) + static_cast<size_t>(slots) * 256 * M, 128);
}
// Work of an item for the deal.  The kernel is bound by the instructions it issues, so a (tile, group)
// weighs what a consumer warp issues for it: about 70 / 73 / 120 / 80 instructions at 1 / 2 / 3 / 4 bits
// (counted in the kernel's loops: one AND per operand register, one MMA per four, the fragment loads and
// the fold).
static unsigned long long item_cost(int tiles_here, const GroupTable& gt, const uint8_t* order, int p0, int p1) {
    static const unsigned kGroupWork[5] = {0, 70, 73, 120, 80};
    unsigned long long w = 0;
    for (int q = p0; q < p1; ++q) w += kGroupWork[gt.bits[order[q]]];
    return w * static_cast<unsigned long long>(tiles_here);
}

static int set_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// First pass over the set: validation of the shapes and everything that depends on all layers.
static int set_geometry(const slim_layer* layers, int n_layers, int g, SetGeometry* sg) {
    if (layers == nullptr || n_layers < 1 || sg == nullptr) return SLIM_ERR_INVALID_ARG;
    memset(sg, 0, sizeof *sg);
    sg->ws_bytes = 256;
    for (int l = 0; l < n_layers; ++l) sg->mmax = sg->mmax > layers[l].M ? sg->mmax : layers[l].M;
    sg->tpw = 2;
    // one token: the 8-bit digit form, 512 bytes per slice; else the tokens of the widest layer rounded up to 8, 16, 32, 64
    sg->mpad = sg->mmax <= 1 ? 2 : (sg->mmax <= 8 ? 8 : (sg->mmax <= 16 ? 16 : (sg->mmax <= 32 ? 32 : 64)));
    const int tpi = kSetConsumers * sg->tpw;          // tiles per item
    for (int l = 0; l < n_layers; ++l) {
        const slim_layer& L = layers[l];
        if (L.M < 1 || L.M > kSetMaxTokens) return SLIM_ERR_INVALID_ARG;
        GroupTable gt;
        const int st = make_group_table(L.N, L.K, g, L.bits_host, &gt);
        if (st != SLIM_OK) return st;
        if (L.N == 0 || L.K == 0) return SLIM_ERR_INVALID_ARG;
        for (int j = 0; j < gt.G; ++j) sg->bmax = sg->bmax > gt.bits[j] ? sg->bmax : gt.bits[j];
        const int items = ((L.N >> 4) + tpi - 1) / tpi;
        sg->n_items += items;
        sg->n_tasks += static_cast<long long>(sg->mpad == 2 ? 1 : sg->mpad) * gt.G;   // staging tasks: (token, group)
        sg->ws_bytes += layer_ws_bytes(sg->mpad, gt);
    }
    if (sg->n_items > 0x3fffffff || sg->n_tasks > 0x3fffffff) return SLIM_ERR_UNSUPPORTED;
    sg->nt = sg->mmax <= 1 ? 1 : sg->mpad / 8;
    // A set with fewer row blocks than persistent CTAs cuts the groups of every row block into parts (items of their
    // own, fp32 partial outputs in the workspace, added in part order by the consumer warp whose part lands last).
    const long long want = static_cast<long long>(set_sm_count()) * (sg->nt >= 4 ? 1 : kSetCtasPerSm);
    sg->split = 1;
    if (sg->n_items < 2 * want) {
        // the number of parts that fills the last wave of CTAs best (the smallest one within 2 % of the best)
        auto items_at = [&](int split) {
            long long n = 0;
            for (int l = 0; l < n_layers; ++l)
                n += static_cast<long long>(layer_split(split, layers[l].K / SLIM_GROUP)) * (((layers[l].N >> 4) + tpi - 1) / tpi);
            return n;
        };
        auto fill = [&](long long n) { return static_cast<double>(n) / static_cast<double>((n + want - 1) / want * want); };
        double best = fill(sg->n_items);
        for (int split = 2; split <= kSetMaxSplit; ++split) {
            const double f = fill(items_at(split));
            if (f > best * 1.02) { best = f; sg->split = split; }
        }
    }
    if (sg->split > 1) {
        sg->n_items = 0;
        long long counters = 0;
        for (int l = 0; l < n_layers; ++l) {
            const slim_layer& L = layers[l];
            const int sp = layer_split(sg->split, L.K / SLIM_GROUP);
            const int n_rb = ((L.N >> 4) + tpi - 1) / tpi;
            sg->n_items += static_cast<long long>(sp) * n_rb;
            if (sp > 1) {
                sg->ws_bytes += align_to(static_cast<size_t>(sp) * L.M * L.N * sizeof(float), 128);
                counters += static_cast<long long>(n_rb) * kSetConsumers;
            }
        }
        if (counters > 65535) return SLIM_ERR_UNSUPPORTED;       // cannot happen: a split set has fewer than 2 x grid row blocks
        sg->n_counters = static_cast<int>(counters);
        sg->cnt_bytes = align_to(static_cast<size_t>(counters) * sizeof(unsigned int), 256);
        sg->ws_bytes += sg->cnt_bytes;
    }
    sg->slot_bytes = static_cast<int>(align_to(static_cast<size_t>(slot_off_w(tpi, sg->mpad)) + static_cast<size_t>(tpi) * 256 * sg->bmax, 128));
    // as many CTAs per SM (kSetCtasPerSm at most) as still leaves each a ring of 4 slots
    const size_t per_sm = 224 * 1024;
    size_t budget = 0;
    for (sg->ctas_per_sm = sg->nt >= 4 ? 1 : kSetCtasPerSm; sg->ctas_per_sm >= 1; --sg->ctas_per_sm) {
        budget = per_sm / sg->ctas_per_sm - 1024 - kSetOffRing;   // 1 KB per CTA is reserved by the system
        if (budget / sg->slot_bytes >= 4 || sg->ctas_per_sm == 1) break;
    }
    size_t slots = budget / sg->slot_bytes;
    if (slots > kSetMaxSlots) slots = kSetMaxSlots;
    if (slots < 2) return SLIM_ERR_UNSUPPORTED;
    sg->n_slots = static_cast<int>(slots);
    sg->smem_bytes = kSetOffRing + slots * sg->slot_bytes;
    long long grid = static_cast<long long>(set_sm_count()) * sg->ctas_per_sm;
    if (grid > kSetMaxGrid) grid = kSetMaxGrid;
    if (grid > sg->n_items) grid = sg->n_items;
    sg->grid = static_cast<int>(grid);
    return SLIM_OK;
}

// Device-side descriptor of one layer.
static void fill_descriptor(const slim_layer& L, const GroupTable& gt, int mpad, int task0, size_t x_off, int split, size_t part_off,
                            int cnt0, SetLayer* out) {
    SetLayer& d = *out;
    memset(&d, 0, sizeof d);
    d.x = static_cast<const __half*>(L.x);
    d.packed = static_cast<const uint8_t*>(L.packed);
    d.scales = static_cast<const __half*>(L.scales);
    d.zeros = static_cast<const __half*>(L.zeros);
    d.y = static_cast<__half*>(L.y);
    d.M = L.M; d.N = L.N; d.K = L.K; d.G = gt.G;
    d.MP = mpad;
    d.task0 = task0;
    d.x_off = x_off;
    d.split = static_cast<uint8_t>(split);
    d.gshift = static_cast<uint8_t>(gt.gshift);
    d.part_off = part_off;
    d.cnt0 = static_cast<uint16_t>(cnt0);
    memcpy(d.prefix, gt.prefix, sizeof d.prefix);
    memcpy(d.bits, gt.bits, sizeof d.bits);
    d.pre3[0] = 0;
    for (int j = 0; j < SLIM_MAX_GROUPS; ++j)
        d.pre3[j + 1] = static_cast<uint16_t>(d.pre3[j] + (j < gt.G && gt.bits[j] == 3 ? 1 : 0));
    int n_sorted = 0;                       // streaming order: by bit-width, then by index
    for (int b = 1; b <= 4; ++b)
        for (int j = 0; j < gt.G; ++j)
            if (gt.bits[j] == b) { d.order[n_sorted++] = static_cast<uint8_t>(j); ++d.count[b - 1]; }
}

static size_t set_plan_bytes(int n_layers, long long n_items) {
    return kSetPlanHeader + static_cast<size_t>(n_layers) * sizeof(SetLayer) + static_cast<size_t>(n_items) * sizeof(SetItem);
}

// Launch configuration with programmatic stream serialization: the kernel may be set up while the one before it in
// the stream is still running; it waits (griddepcontrol.wait) before it touches what that kernel reads or writes.
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    PdlLaunch(unsigned grid, unsigned block, size_t smem, cudaStream_t stream, bool early = true) {
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(grid, 1, 1);
        cfg.blockDim = dim3(block, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = early ? 1 : 0;
    }
};

template <int NT, bool ONE, int TPW>
static cudaError_t launch_set(const SetParams& prm, int grid, size_t smem, cudaStream_t stream, bool early) {
    static std::atomic<bool> attr_set[64];    // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemv_set_kernel<NT, ONE, TPW>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    PdlLaunch l(static_cast<unsigned>(grid), kSetThreads, smem, stream, early);
    return cudaLaunchKernelEx(&l.cfg, gemv_set_kernel<NT, ONE, TPW>, prm);
}

}  // namespace slim

namespace slim {

// ------------------------------------------------------------------------------------------ large single layers through the ring
// A layer of kRouteMinBytes or more is enough work for the persistent kernel on its own (its row blocks cut into parts
// when they are fewer than the CTAs), and a launch per layer of the cluster kernel reaches a third of that rate on it.
constexpr size_t kRouteMinBytes = 32u << 20;

struct RouteLayout {
    SetGeometry sg;
    int n_rb, sp;
    size_t plan_off, plan_bytes, x_off, part_off, total;
};

static bool route_layout(int M, int N, int K, int g, const uint8_t* bits_host, const GroupTable& gt, RouteLayout* r) {
    if (M < 1 || N <= 0 || static_cast<size_t>(16) * N * gt.prefix[gt.G] < kRouteMinBytes) return false;
    slim_layer L;
    memset(&L, 0, sizeof L);
    L.bits_host = bits_host; L.M = M; L.N = N; L.K = K;
    if (set_geometry(&L, 1, g, &r->sg) != SLIM_OK) return false;
    const int tpi = kSetConsumers * r->sg.tpw;
    r->n_rb = ((N >> 4) + tpi - 1) / tpi;
    r->sp = layer_split(r->sg.split, gt.G);
    r->plan_off = kSetOffCounters + r->sg.cnt_bytes;
    r->plan_bytes = set_plan_bytes(1, static_cast<long long>(r->n_rb) * r->sp);
    r->x_off = r->plan_off + align_to(r->plan_bytes, 256);
    r->part_off = r->x_off + layer_ws_bytes(r->sg.mpad, gt);
    r->total = r->part_off + (r->sp > 1 ? align_to(static_cast<size_t>(r->sp) * M * N * sizeof(float), 128) : 0);
    return true;
}

size_t gemv_route_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, const GroupTable& gt) {
    RouteLayout r;
    return route_layout(M, N, K, g, bits_host, gt, &r) ? r.total : 0;
}

}  // namespace slim

namespace slim {

// Checks a launch record and fills the kernel parameters and the dynamic shared memory of the persistent kernel.
static int set_params(const slim_gemv_set_info* info, const void* plan, void* workspace, size_t workspace_bytes, SetParams* out, size_t* smem_out) {
    if (info == nullptr || plan == nullptr) return SLIM_ERR_INVALID_ARG;
    if (info->n_layers < 1 || info->grid < 1 || info->grid > kSetMaxGrid || info->n_slots < 2 ||
        info->n_slots > kSetMaxSlots || info->slot_bytes < 128 || info->slot_bytes % 128 != 0 ||
        (info->token_tiles != 1 && info->token_tiles != 2 && info->token_tiles != 4 && info->token_tiles != 8) ||
        info->max_tokens < 1 || info->max_tokens > 8 * info->token_tiles ||
        info->tiles_per_warp != 2 ||
        info->max_bits < 1 || info->max_bits > 4 || info->stage_tasks < 1 || info->split < 1 || info->split > kSetMaxSplit ||
        info->n_counters < 0 || info->n_counters > 65535 || info->n_layers > 65535)
        return SLIM_ERR_INVALID_ARG;
    const size_t smem = kSetOffRing + static_cast<size_t>(info->n_slots) * info->slot_bytes;
    if (smem > 224 * 1024) return SLIM_ERR_INVALID_ARG;
    if (!aligned16(plan)) return SLIM_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < info->workspace_bytes || workspace_bytes < 256 ||
        workspace_bytes < kSetOffCounters + static_cast<size_t>(info->n_counters) * sizeof(unsigned int))
        return SLIM_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
    SetParams& prm = *out;
    memset(&prm, 0, sizeof prm);
    prm.item_begin = static_cast<const int*>(plan);
    prm.layers = reinterpret_cast<const SetLayer*>(static_cast<const uint8_t*>(plan) + kSetPlanHeader);
    prm.items = reinterpret_cast<const SetItem*>(prm.layers + info->n_layers);
    prm.ws = static_cast<uint8_t*>(workspace);
    prm.n_layers = info->n_layers;
    prm.n_slots = info->n_slots;
    prm.slot_bytes = info->slot_bytes;
    prm.one = 1;
    const int tpi = kSetConsumers * info->tiles_per_warp;
    const int mp = info->max_tokens == 1 ? 2 : 8 * info->token_tiles;
    if (slot_off_w(tpi, mp) + tpi * 256 * info->max_bits > info->slot_bytes) return SLIM_ERR_INVALID_ARG;
    *smem_out = smem;
    return SLIM_OK;
}

// The persistent kernel of the set in the form its token count asks for.
static int launch_set_for(const slim_gemv_set_info* info, const SetParams& prm, size_t smem, cudaStream_t s, bool early) {
    const cudaError_t e = info->max_tokens == 1 ? launch_set<1, true, 2>(prm, info->grid, smem, s, early)
                        : info->token_tiles == 8 ? launch_set<8, false, 2>(prm, info->grid, smem, s, early)
                        : info->token_tiles == 4 ? launch_set<4, false, 2>(prm, info->grid, smem, s, early)
                        : info->token_tiles == 1 ? launch_set<1, false, 2>(prm, info->grid, smem, s, early)
                                                 : launch_set<2, false, 2>(prm, info->grid, smem, s, early);
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

// Returns SLIM_OK after enqueueing the layer through the layer-set kernels, a negative status on failure, or 1 if this
// shape or workspace is not routed (the caller then takes the per-layer kernel).
int gemv_route(const void* x, const void* packed, const uint8_t* bits_host, const GroupTable& gt, const void* scales, const void* zeros,
               void* y, int M, int N, int K, int g, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    RouteLayout r;
    if (!route_layout(M, N, K, g, bits_host, gt, &r) || workspace_bytes < r.total) return 1;
    slim_layer L;
    memset(&L, 0, sizeof L);
    L.x = x; L.packed = packed; L.scales = scales; L.zeros = zeros; L.y = y; L.bits_host = bits_host; L.M = M; L.N = N; L.K = K;
    SetLayer d;
    fill_descriptor(L, gt, r.sg.mpad, 0, r.x_off, r.sp, r.part_off, 0, &d);
    uint8_t* plan = static_cast<uint8_t*>(workspace) + r.plan_off;
    const long long n_items = static_cast<long long>(r.n_rb) * r.sp;
    const int grid = static_cast<int>(n_items < r.sg.grid ? n_items : r.sg.grid);
    slim_gemv_set_info info;
    memset(&info, 0, sizeof info);
    info.n_layers = 1;
    info.grid = grid;
    info.n_slots = r.sg.n_slots;
    info.slot_bytes = r.sg.slot_bytes;
    info.token_tiles = r.sg.nt;
    info.stage_tasks = (r.sg.mpad == 2 ? 1 : r.sg.mpad) * gt.G;
    info.n_items = static_cast<int>(n_items);
    info.max_bits = r.sg.bmax;
    info.max_tokens = r.sg.mmax;
    info.tiles_per_warp = r.sg.tpw;
    info.split = r.sg.split;
    info.n_counters = r.sg.n_counters;
    info.plan_bytes = r.plan_bytes;
    info.workspace_bytes = r.total;
    SetParams prm;
    size_t smem = 0;
    const int st = set_params(&info, plan, workspace, workspace_bytes, &prm, &smem);
    if (st != SLIM_OK) return st;
    // One token: both kernels are launched early (the staging kernel is a handful of blocks).  With more tokens its
    // blocks are many and early launches measured 1 to 4 % slower, so those keep plain stream order.
    const bool early = M == 1;
    {
        PdlLaunch l(static_cast<unsigned>((info.stage_tasks + 7) / 8), 256, 0, stream, early);
        SLIM_CUDA_TRY(cudaLaunchKernelEx(&l.cfg, set_single_stage_kernel, d, plan, prm.ws, grid, r.n_rb, r.sp, info.stage_tasks, info.n_counters));
    }
    return launch_set_for(&info, prm, smem, stream, early);
}

}  // namespace slim

extern "C" {

int slim_gemv_set_bytes(const slim_layer* layers_host, int n_layers, int g, size_t* plan_bytes, size_t* workspace_bytes) {
    if (plan_bytes == nullptr || workspace_bytes == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::SetGeometry sg;
    const int st = slim::set_geometry(layers_host, n_layers, g, &sg);
    if (st != SLIM_OK) return st;
    *plan_bytes = slim::set_plan_bytes(n_layers, sg.n_items);
    *workspace_bytes = sg.ws_bytes;
    return SLIM_OK;
}

int slim_gemv_set_plan(const slim_layer* layers_host, int n_layers, int g, void* plan, size_t plan_bytes,
                       slim_gemv_set_info* info, void* stream) {
    if (info == nullptr || plan == nullptr) return SLIM_ERR_INVALID_ARG;
    slim::SetGeometry sg;
    const int st = slim::set_geometry(layers_host, n_layers, g, &sg);
    if (st != SLIM_OK) return st;
    if (!slim::aligned16(plan)) return SLIM_ERR_ALIGNMENT;
    if (plan_bytes < slim::set_plan_bytes(n_layers, sg.n_items)) return SLIM_ERR_WORKSPACE;
    for (int l = 0; l < n_layers; ++l) {
        const slim_layer& L = layers_host[l];
        if (L.x == nullptr || L.packed == nullptr || L.scales == nullptr || L.zeros == nullptr || L.y == nullptr)
            return SLIM_ERR_INVALID_ARG;
        if (!slim::aligned16(L.x) || !slim::aligned16(L.packed) || !slim::aligned16(L.scales) || !slim::aligned16(L.zeros) ||
            !slim::aligned16(L.y))
            return SLIM_ERR_ALIGNMENT;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* plan_dev = static_cast<uint8_t*>(plan);

    try {                       // the host-side lists may fail to allocate: reported as a status
    // A single-token set small enough for all its CTAs to be resident at once runs as one launch without a ring.
    if (sg.mmax == 1) {
        slim::OneSetPlan op;
        const int taken = slim::one_set_plan(layers_host, n_layers, g, plan, plan_bytes, s, &op);
        if (taken < 0) return taken;
        if (taken == SLIM_OK) {
            memset(info, 0, sizeof *info);
            info->n_layers = n_layers;
            info->grid = op.grid;
            info->token_tiles = 1;
            info->max_bits = sg.bmax;
            info->max_tokens = 1;
            info->tiles_per_warp = 2;
            info->split = 1;
            info->n_items = op.grid;
            info->resident_pairs = op.pairs;
            info->resident_cluster = op.cluster;
            info->resident_smem = op.smem;
            info->plan_bytes = slim::set_plan_bytes(n_layers, sg.n_items);
            info->workspace_bytes = 256;
            return SLIM_OK;
        }
    }
    // Second pass: descriptors and items.  The copies below read host memory that goes out of scope:
    // pageable sources are staged before cudaMemcpyAsync returns.
    static_assert((slim::kSetMaxGrid + 1) * sizeof(int) <= slim::kSetPlanHeader, "item ranges fit the plan header");
    std::vector<slim::SetItem> items;
    std::vector<unsigned long long> cost;
    items.reserve(static_cast<size_t>(sg.n_items));
    cost.reserve(static_cast<size_t>(sg.n_items));
    const int tpi = slim::kSetConsumers * sg.tpw;
    int task = 0, cnt0 = 0;
    size_t ws_off = slim::kSetOffCounters + sg.cnt_bytes;
    // workspace: header, the arrival counters of the split row blocks, the staged activations of all layers, then the
    // fp32 partial outputs of the layers that are split
    std::vector<size_t> part_off(static_cast<size_t>(n_layers), 0), x_off(static_cast<size_t>(n_layers), 0);
    {
        size_t off = ws_off;
        for (int l = 0; l < n_layers; ++l) {
            slim::GroupTable gt;
            slim::make_group_table(layers_host[l].N, layers_host[l].K, g, layers_host[l].bits_host, &gt);
            off += slim::layer_ws_bytes(sg.mpad, gt);
        }
        for (int l = 0; l < n_layers; ++l) {
            const slim_layer& L = layers_host[l];
            const int sp = slim::layer_split(sg.split, L.K / SLIM_GROUP);
            part_off[l] = off;
            if (sp > 1) off += slim::align_to(static_cast<size_t>(sp) * L.M * L.N * sizeof(float), 128);
        }
    }
    for (int l = 0; l < n_layers; ++l) {
        const slim_layer& L = layers_host[l];
        slim::GroupTable gt;
        slim::make_group_table(L.N, L.K, g, L.bits_host, &gt);
        slim::SetLayer d;
        const int sp = slim::layer_split(sg.split, gt.G);
        // A layer that reads the activations of an earlier layer through the same bit map (the staged form depends
        // on the group's bit-width) uses that layer's staged copy and has no staging tasks of its own.
        int same = -1;
        for (int e = 0; e < l && same < 0; ++e) {
            const slim_layer& E = layers_host[e];
            if (E.x == L.x && E.M == L.M && E.K == L.K && memcmp(E.bits_host, L.bits_host, static_cast<size_t>(L.K / g)) == 0) same = e;
        }
        x_off[l] = same >= 0 ? x_off[same] : ws_off;
        slim::fill_descriptor(L, gt, sg.mpad, task, x_off[l], sp, part_off[l], cnt0, &d);
        ws_off += slim::layer_ws_bytes(sg.mpad, gt);
        SLIM_CUDA_TRY(cudaMemcpyAsync(plan_dev + slim::kSetPlanHeader + static_cast<size_t>(l) * sizeof d, &d, sizeof d,
                                      cudaMemcpyHostToDevice, s));
        const int n_rb = ((L.N >> 4) + tpi - 1) / tpi;
        if (sp > 1) cnt0 += n_rb * slim::kSetConsumers;
        for (int rb = 0; rb < n_rb; ++rb) {
            const int th = (L.N >> 4) - tpi * rb;
            for (int part = 0; part < sp; ++part) {
                const int p0 = gt.G * part / sp, p1 = gt.G * (part + 1) / sp;
                slim::SetItem it;
                memset(&it, 0, sizeof it);
                it.layer = l; it.rb = rb; it.N = L.N; it.range = p0 | (p1 << 16); it.M = L.M;
                it.counts = d.count[0] | (d.count[1] << 9) | (d.count[2] << 18);
                if (sp > 1) {      // its fp32 partial output [M][N], as a workspace offset
                    it.y = reinterpret_cast<__half*>(part_off[l] + static_cast<size_t>(part) * L.M * L.N * sizeof(float));
                    it.counts |= slim::kItemPartial;
                } else {
                    it.y = d.y;
                }
                items.push_back(it);
                cost.push_back(slim::item_cost(th < tpi ? th : tpi, gt, d.order, p0, p1));
            }
        }
        if (same < 0) task += (sg.mpad == 2 ? 1 : sg.mpad) * gt.G;
    }
    // The deal: items by falling cost (equal costs in the set's order), each to the CTA that has the
    // least so far (the lowest-numbered of equals).  Within a CTA the heavy items come first.
    const int n_items = static_cast<int>(items.size());
    std::vector<int> by_cost(n_items);
    for (int i = 0; i < n_items; ++i) by_cost[i] = i;
    std::stable_sort(by_cost.begin(), by_cost.end(), [&](int a, int b) { return cost[a] > cost[b]; });
    typedef std::pair<unsigned long long, int> Load;                 // (work so far, CTA)
    std::priority_queue<Load, std::vector<Load>, std::greater<Load> > least;
    for (int c = 0; c < sg.grid; ++c) least.push(Load(0ull, c));
    std::vector<int> owner(n_items), count(sg.grid + 1, 0);
    for (int k = 0; k < n_items; ++k) {
        Load top = least.top();
        least.pop();
        owner[by_cost[k]] = top.second;
        ++count[top.second + 1];
        least.push(Load(top.first + cost[by_cost[k]], top.second));
    }
    int item_begin[slim::kSetMaxGrid + 1];
    item_begin[0] = 0;
    for (int c = 0; c < sg.grid; ++c) item_begin[c + 1] = item_begin[c] + count[c + 1];
    std::vector<slim::SetItem> dealt(n_items);
    std::vector<int> fill(item_begin, item_begin + sg.grid);
    for (int k = 0; k < n_items; ++k) dealt[fill[owner[by_cost[k]]]++] = items[by_cost[k]];
    SLIM_CUDA_TRY(cudaMemcpyAsync(plan_dev, item_begin, static_cast<size_t>(sg.grid + 1) * sizeof(int), cudaMemcpyHostToDevice, s));
    SLIM_CUDA_TRY(cudaMemcpyAsync(plan_dev + slim::kSetPlanHeader + static_cast<size_t>(n_layers) * sizeof(slim::SetLayer), dealt.data(),
                                  static_cast<size_t>(n_items) * sizeof(slim::SetItem), cudaMemcpyHostToDevice, s));
    const int item = n_items;

    memset(info, 0, sizeof *info);
    info->n_layers = n_layers;
    info->grid = sg.grid;
    info->n_slots = sg.n_slots;
    info->slot_bytes = sg.slot_bytes;
    info->token_tiles = sg.nt;
    info->stage_tasks = task;
    info->n_items = item;
    info->max_bits = sg.bmax;
    info->max_tokens = sg.mmax;
    info->tiles_per_warp = sg.tpw;
    info->split = sg.split;
    info->n_counters = sg.n_counters;
    info->plan_bytes = slim::set_plan_bytes(n_layers, n_items);
    info->workspace_bytes = sg.ws_bytes;
    } catch (const std::exception&) {
        return SLIM_ERR_UNSUPPORTED;
    }
    return SLIM_OK;
}


int slim_selftest_wait_timeout(void* workspace, size_t workspace_bytes, unsigned int limit_us, void* stream) {
    if (workspace == nullptr || workspace_bytes < 256) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
    if (limit_us < 1 || limit_us > 100000) return SLIM_ERR_INVALID_ARG;
    slim::wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint8_t*>(workspace),
                                                                               1000ull * limit_us);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int slim_mpq_gemv_set(const slim_gemv_set_info* info, const void* plan, void* workspace, size_t workspace_bytes, void* stream) {
    if (info != nullptr && info->resident_pairs > 0) {
        if (plan == nullptr) return SLIM_ERR_INVALID_ARG;
        if (!slim::aligned16(plan)) return SLIM_ERR_ALIGNMENT;
        if (workspace == nullptr || workspace_bytes < 256) return SLIM_ERR_WORKSPACE;
        if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
        slim::OneSetPlan op;
        op.pairs = info->resident_pairs; op.cluster = info->resident_cluster; op.grid = info->grid; op.smem = info->resident_smem;
        return slim::one_set_launch(op, plan, info->n_layers, workspace, static_cast<cudaStream_t>(stream));
    }
    slim::SetParams prm;
    size_t smem = 0;
    const int st = slim::set_params(info, plan, workspace, workspace_bytes, &prm, &smem);
    if (st != SLIM_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        slim::PdlLaunch l(static_cast<unsigned>((info->stage_tasks + 7) / 8), 256, 0, s, false);
        SLIM_CUDA_TRY(cudaLaunchKernelEx(&l.cfg, slim::gemv_set_stage_kernel, prm.layers, prm.ws, info->n_layers, info->stage_tasks, info->n_counters));
    }
    return slim::launch_set_for(info, prm, smem, s, false);
}

}  // extern "C"
