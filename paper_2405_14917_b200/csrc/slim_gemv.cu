// slim_mpq_gemv: decode path (1 <= M <= 16) of the mixed-precision linear layer, sm_100a.
//
// The kernel streams the packed slices exactly once (HBM-bound) and does the dot products on
// the tensor cores (mma.sync m16n8k16, fp16 x fp16 -> fp32) without materialising fp16 weights:
//
//  * A operand = raw code slices.  A 16-bit half whose exponent and sign bits are zero and whose
//    mantissa holds a code field v at bit position pos is the subnormal v * 2^(pos-24), exactly.
//    A slice word keeps the fields of columns f and f + nf/2 sixteen bits apart, so ONE AND
//    yields a ready-to-use half2 operand (two weights); fields above mantissa bit 9 need the word
//    shifted right once first.
//  * B operand = activations, staged once per CTA in fragment order: x[m][k] * 2^(S + lo - pos),
//    where pos undoes the field position of the weight it will meet, lo is the slice's offset
//    inside the code, and 2^S (per token and group, from max|x|) lifts the values to the top of the
//    fp16 range so that the small ones keep their bits.
//  * The MMA accumulates the exact products in fp32.  Per (row, group) the group partial D is
//    folded as acc += s * (D * 2^(24-S) - z * sum_k x_k), which is s * sum_k x_k (q_k - z).
//
// Work split.  A layer is smaller than, or comparable to, the bytes HBM must keep in flight, and
// a warp's instruction stream is the critical path, so the kernel spreads a layer over as many
// warps as possible and is built around latency:
//  * grid = (CS k-slices) x (row blocks of T 16-row tiles); the CS CTAs of one row block form a
//    thread-block cluster.  Warp w of a CTA owns tile w % T and takes every (8/T)-th group of the
//    CTA's range, so x is staged once for T tiles; the range is walked in chunks of GC groups
//    (one chunk for decode-sized inputs).
//  * Every warp issues the weight, scale and zero bytes of its groups of the first chunk as
//    16-byte cp.async copies in its first instructions; chunk c+1 is in flight while chunk c is
//    consumed.
//  * The kernel is launched with programmatic stream serialisation: it lets the next kernel
//    start at once (whose copies then overlap this kernel's arithmetic) and waits for the
//    previous kernel only before it touches x or y.
//  * x is put into B-fragment order by one warp per (token, group), which also finds the group's
//    max |x| and sum with shuffles: one barrier between landing and use.
//  * Partial sums are added across warps in shared memory; across the cluster every CTA owns a
//    share of the outputs, receives the other CTAs' partials for it through distributed shared
//    memory and adds them in rank order (deterministic); no global scratch.
#include "slim_gemv_dev.cuh"

#include <atomic>

#include <cstring>

namespace slim {

constexpr int kMaxWarps = 8;
constexpr int kMaxCluster = 8;
constexpr int kWsHeader = 256;              // status word + padding
constexpr int kPreStageMinM = 4;            // from this many tokens on, x is put into fragment order by a kernel of its own

struct GemvParams {
    const __half* x;
    const uint8_t* packed;
    const __half* scales;
    const __half* zeros;
    __half* y;
    const uint8_t* xs_g;    // pre-staged B fragments [slot][8 mma][M][4 lanes] x 8 B (pre-staged mode)
    const float2* sxe_g;    // pre-staged (sum_k x, 2^(24-S)) [G][16] (pre-staged mode)
    int M, N, K;
    int CS;                 // k-slices (= cluster size)
    int W;                  // warps per CTA
    int T;                  // 16-row tiles per CTA (divides W)
    int GC;                 // groups per chunk
    int region_bytes;       // landing buffer of one chunk (largest chunk, all T tiles)
    int max_slots;          // most slices in any chunk
    int two_bufs;           // some k-slice has more than one chunk: weights and raw x are double-buffered
    uint16_t kbegin[kMaxCluster + 1];
    uint16_t pre3[SLIM_MAX_GROUPS + 1];   // pre3[j] = number of 3-bit groups (two slices) before group j
    GroupTable gt;
};

// ------------------------------------------------------------------------------------------ shared memory map
struct SmemMap {
    uint32_t sxe;      // float2[GC][16]: (sum_k x, 2^(24-S)) per (group, token)
    uint32_t red;      // float[W][M][16]: per-warp partial outputs
    uint32_t cred;     // float2[CS][share]: partial outputs received from the cluster's CTAs
    uint32_t xraw;     // half[2][M][GC*128] (double-buffered)
    uint32_t xs;       // [slots][8 mma][M tokens][4 lanes] x 8 B: B fragments
    uint32_t wbuf;     // [2][region_bytes]: packed slices, scales, zeros of the chunk
    uint32_t total;
};
__host__ __device__ inline uint32_t align_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }
// Output pairs (two rows of one token) a CTA owns in the cluster reduction.
__host__ __device__ inline int cluster_share(int T, int M, int CS) { return (T * M * 8 + CS - 1) / CS; }
// `pre`: x arrives already in fragment order (no raw x; fragments and sums double-buffered instead).
__host__ __device__ inline SmemMap make_smem_map(int M, int W, int T, int CS, int GC, int region_bytes, int max_slots, bool two_bufs,
                                                 bool pre) {
    SmemMap m;
    uint32_t o = 0;
    m.sxe = o;   o += (pre && two_bufs ? 2u : 1u) * 128u * GC;
    m.red = o;   o += 64u * W * M;
    m.cred = o;  o += CS > 1 ? 8u * CS * cluster_share(T, M, CS) : 0u;
    o = align_up(o, 16);
    m.xraw = o;  o += pre ? 0u : (two_bufs ? 2u : 1u) * (256u * M * GC);
    o = align_up(o, 128);
    m.xs = o;    o += (pre && two_bufs ? 2u : 1u) * static_cast<uint32_t>(max_slots) * 8 * M * 32;
    o = align_up(o, 128);
    m.wbuf = o;  o += (two_bufs ? 2u : 1u) * region_bytes;
    m.total = o;
    return m;
}

// ------------------------------------------------------------------------------------------ kernels
// Pre-staging kernel (M >= kPreStageMinM): one warp per (token, group) writes the fragments and
// sums of the whole x to global scratch once, instead of every row block repeating the work.
struct StageParams {
    const __half* x;
    uint8_t* xs_g;
    float2* sxe_g;
    int M, K, G;
    uint16_t pre3[SLIM_MAX_GROUPS + 1];
    uint8_t bits[SLIM_MAX_GROUPS];
};
__global__ void __launch_bounds__(256) gemv_stage_x_kernel(const __grid_constant__ StageParams p) {
    pdl_launch_dependents();
    pdl_wait();                                          // x may come from the previous kernel
    const int lane = threadIdx.x & 31;
    const int pi = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (pi >= p.M * p.G) return;
    const int m = pi / p.G, j = pi - m * p.G;
    const float2 r = stage_group(p.x + static_cast<size_t>(m) * p.K + j * SLIM_GROUP,
                                 p.xs_g + static_cast<size_t>(j + p.pre3[j]) * 8 * p.M * 32, p.bits[j], m, p.M, lane);
    if (lane == 0) p.sxe_g[j * 16 + m] = r;
    if (m == 0 && lane < 16 && lane >= p.M) p.sxe_g[j * 16 + lane] = make_float2(0.f, 1.f);   // absent tokens read 0
}

template <int NT, bool PRE>   // NT 8-token MMA tiles: 1 (M <= 8) or 2; PRE: x arrives pre-staged
__global__ void __launch_bounds__(kMaxWarps * 32) gemv_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    // Let the next kernel of the stream start at once: it only prefetches its own weights until
    // this kernel has finished.
    pdl_launch_dependents();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int W = p.W, T = p.T, KW = W / T, nthreads = W * 32;
    const int gq = lane >> 2, c = lane & 3;
    const int ks = blockIdx.x, rb = blockIdx.y;
    const int N = p.N, M = p.M, GC = p.GC;
    const int g0 = p.kbegin[ks], g1 = p.kbegin[ks + 1];
    const int ng = g1 - g0;
    const int n_chunks = (ng + GC - 1) / GC;
    const SmemMap sm = make_smem_map(M, W, T, p.CS, GC, p.region_bytes, p.max_slots, p.two_bufs != 0, PRE);
    const uint32_t xs_stride = static_cast<uint32_t>(p.max_slots) * 8 * M * 32;   // bytes per fragment buffer (pre-staged mode)
    const uint32_t xraw_stride = 256u * M * GC;                   // bytes per xraw buffer
    const int tw = warp % T, kw = warp / T;                       // this warp's tile of the CTA and k-way
    const int tile = rb * T + tw;
    const bool active = tile < (N >> 4);

    // Layout of a chunk buffer: group after group, inside a group the T tiles one after another,
    // each as its slices followed by 32 bytes of scales and 32 bytes of zeros.
    auto item_addr = [&](uint32_t buf, int ja, int j, int b) -> uint32_t {
        return buf + T * (256u * (p.gt.prefix[j] - p.gt.prefix[ja]) + 64u * (j - ja)) + tw * (256u * b + 64u);
    };
    // weights, scales and zeros of this warp's items of chunk `ch` -> buffer ch & 1
    auto issue_weights = [&](int ch) {
        if (active && ch < n_chunks) {
            const int ja = g0 + ch * GC, jb = min(g1, ja + GC);
            const uint32_t buf = sbase + sm.wbuf + (ch & 1) * p.region_bytes;
            for (int j = ja + kw; j < jb; j += KW) {
                const int b = p.gt.bits[j];
                const uint32_t dst = item_addr(buf, ja, j, b);
                const uint8_t* src = p.packed + 16ull * N * p.gt.prefix[j] + static_cast<size_t>(tile) * 256 * b;
                if (lane < 16 * b) cp_async16(dst + 16 * lane, src + 16 * lane);
                if (lane + 32 < 16 * b) cp_async16(dst + 16 * (lane + 32), src + 16 * (lane + 32));
                if (lane < 4) {
                    const __half* sz = (lane < 2 ? p.scales : p.zeros) + static_cast<size_t>(j >> p.gt.gshift) * N + 16 * tile + 8 * (lane & 1);
                    cp_async16(dst + 256 * b + 16 * lane, sz);
                }
            }
        }
        cp_async_commit();
    };
    // raw activations of chunk `ch` (all tokens) -> xraw buffer ch & 1
    auto issue_x = [&](int ch) {
        if (PRE && ch < n_chunks) {
            // fragments and sums of the chunk, already in their final order
            const int ja = g0 + ch * GC, jb = min(g1, ja + GC);
            const int s0 = ja + p.pre3[ja], s1 = jb + p.pre3[jb];
            const int n16 = (s1 - s0) * 16 * M;                            // 16-byte pieces of the fragments
            const uint32_t dst = sbase + sm.xs + (ch & 1) * xs_stride;
            const uint8_t* src = p.xs_g + static_cast<size_t>(s0) * 8 * M * 32;
            for (int q = tid; q < n16; q += nthreads) cp_async16(dst + 16 * q, src + 16 * q);
            const uint32_t dsx = sbase + sm.sxe + (ch & 1) * 128u * GC;
            for (int q = tid; q < (jb - ja) * 8; q += nthreads)
                cp_async16(dsx + 16 * q, reinterpret_cast<const uint8_t*>(p.sxe_g + ja * 16) + 16 * q);
        } else if (ch < n_chunks) {
            const int ja = g0 + ch * GC, cg = min(g1, ja + GC) - ja;
            const int per_tok = cg * 16;                                   // 16-byte pieces per token
            const uint32_t dst0 = sbase + sm.xraw + (ch & 1) * xraw_stride;
            for (int m = 0; m < M; ++m)
                for (int q = tid; q < per_tok; q += nthreads)
                    cp_async16(dst0 + (m * GC * SLIM_GROUP + 8 * q) * 2, p.x + static_cast<size_t>(m) * p.K + ja * SLIM_GROUP + 8 * q);
        }
        cp_async_commit();
    };

    // ---- put the first chunk in flight, then wait until the previous kernel has finished before
    // x or y are touched
    issue_weights(0);
    if (p.CS > 1) cluster_arrive_relaxed();          // "this CTA runs": awaited before the first store into a peer's shared memory
    pdl_wait();
    issue_x(0);
    if (!PRE)
        for (int i = tid; i < 32 * GC; i += nthreads) reinterpret_cast<float*>(smem + sm.sxe)[i] = 0.f;   // absent tokens read 0

    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[n][r] = 0.f;

    for (int ch = 0; ch < n_chunks; ++ch) {
        const int ja = g0 + ch * GC, cg = min(g1, ja + GC) - ja;
        const int kc = GC * SLIM_GROUP;                                   // xraw row stride (halves)
        const __half* xraw = reinterpret_cast<const __half*>(smem + sm.xraw + (ch & 1) * xraw_stride);
        float2* sxe = reinterpret_cast<float2*>(smem + sm.sxe + (PRE ? (ch & 1) * 128u * GC : 0u));
        const uint32_t xs_buf = sbase + sm.xs + (PRE ? (ch & 1) * xs_stride : 0u);

        cp_async_wait_all();             // x and weights of this chunk have landed (this thread's copies)
        __syncthreads();                 // ... everybody's; and the previous chunk is fully consumed
        issue_weights(ch + 1);           // into the buffer the previous chunk has left
        if (PRE) {
            issue_x(ch + 1);             // its fragments and sums too
        } else {
            // ---- activations in B-fragment order: one warp per (token, group) --------------------------
            for (int pi = warp; pi < M * cg; pi += W) {
                const int m = pi / cg, i = pi - m * cg;
                const int slot0 = i + p.pre3[ja + i] - p.pre3[ja];
                const float2 r = stage_group(xraw + m * kc + i * SLIM_GROUP, smem + sm.xs + static_cast<size_t>(slot0) * 8 * M * 32,
                                             p.gt.bits[ja + i], m, M, lane);
                if (lane == 0) sxe[i * 16 + m] = r;
            }
            issue_x(ch + 1);
            __syncthreads();
        }

        // ---- this warp's tile against its groups of the chunk --------------------------------------------
        if (active) {
            const uint32_t buf = sbase + sm.wbuf + (ch & 1) * p.region_bytes;
            for (int it = kw; it < cg; it += KW) {
                const int b = p.gt.bits[ja + it];
                const uint32_t item = item_addr(buf, ja, ja + it, b);
                const uint32_t xs_slot0 = xs_buf + static_cast<uint32_t>(it + p.pre3[ja + it] - p.pre3[ja]) * 8 * M * 32;

                float d[2][NT][4];       // two interleaved accumulation chains
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int n = 0; n < NT; ++n)
#pragma unroll
                        for (int r = 0; r < 4; ++r) d[h][n][r] = 0.f;

                // one slice of width WD starting at unit `unit0`, activations in staging slot `xs_slot`
                auto run_slice = [&](auto wtag, int unit0, uint32_t xs_slot) {
                    constexpr int WD = decltype(wtag)::value;
                    constexpr int MPU = 8 / WD;                 // MMAs per unit
#pragma unroll
                    for (int u = 0; u < WD; ++u) {
                        const uint2 wd = lds64(item + 256 * (unit0 + u) + 8 * lane);
                        const uint32_t shx = wd.x >> pair_shift(WD), shy = wd.y >> pair_shift(WD);
#pragma unroll
                        for (int ii = 0; ii < MPU; ++ii) {
                            const uint32_t a0 = pair<WD>(wd.x, shx, 2 * ii), a1 = pair<WD>(wd.y, shy, 2 * ii);
                            const uint32_t a2 = pair<WD>(wd.x, shx, 2 * ii + 1), a3 = pair<WD>(wd.y, shy, 2 * ii + 1);
                            const int mi = u * MPU + ii;
#pragma unroll
                            for (int n = 0; n < NT; ++n) {
                                const int m = 8 * n + gq;
                                uint2 bv = make_uint2(0u, 0u);
                                if (m < M) bv = lds64(xs_slot + ((mi * M + m) * 4 + c) * 8);
                                mma_f16(d[ii & 1][n], a0, a1, a2, a3, bv);
                            }
                        }
                    }
                };
                switch (b) {
                    case 1: run_slice(W1{}, 0, xs_slot0); break;
                    case 2: run_slice(W2{}, 0, xs_slot0); break;
                    case 3: run_slice(W2{}, 0, xs_slot0); run_slice(W1{}, 2, xs_slot0 + 8 * M * 32); break;
                    default: run_slice(W4{}, 0, xs_slot0); break;
                }

                // fold the group: acc += s * (D * 2^(24-S) - z * sum_x); rows 2gq, 2gq+1, tokens 8n+2c, 8n+2c+1
                const uint32_t s2 = lds32(item + 256 * b + gq * 4);
                const uint32_t z2 = lds32(item + 256 * b + 32 + gq * 4);
                const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
                const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&z2));
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    const float4 t = *reinterpret_cast<const float4*>(sxe + it * 16 + 8 * n + 2 * c);   // (sx0, e0, sx1, e1)
                    const float d0 = (d[0][n][0] + d[1][n][0]) * t.y, d1 = (d[0][n][1] + d[1][n][1]) * t.w;
                    const float d2 = (d[0][n][2] + d[1][n][2]) * t.y, d3 = (d[0][n][3] + d[1][n][3]) * t.w;
                    acc[n][0] = fmaf(sf.x, fmaf(-zf.x, t.x, d0), acc[n][0]);
                    acc[n][1] = fmaf(sf.x, fmaf(-zf.x, t.z, d1), acc[n][1]);
                    acc[n][2] = fmaf(sf.y, fmaf(-zf.y, t.x, d2), acc[n][2]);
                    acc[n][3] = fmaf(sf.y, fmaf(-zf.y, t.z, d3), acc[n][3]);
                }
            }
        }
    }

    // ---- add the partial sums of the warps that share a tile (fixed order) ---------------------------
    float* red = reinterpret_cast<float*>(smem + sm.red);      // [W][M][16], warp = kw * T + tw
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const int m0 = 8 * n + 2 * c;
        if (m0 < M) *reinterpret_cast<float2*>(red + (warp * M + m0) * 16 + 2 * gq) = make_float2(acc[n][0], acc[n][2]);
        if (m0 + 1 < M) *reinterpret_cast<float2*>(red + (warp * M + m0 + 1) * 16 + 2 * gq) = make_float2(acc[n][1], acc[n][3]);
    }
    __syncthreads();
    const int CS = p.CS;
    const int pairs = T * M * 8;                                // e = (tile of the CTA, token, row pair)
    const int share = cluster_share(T, M, CS);
    const uint32_t rank = CS > 1 ? cluster_ctarank() : 0u;
    auto store_out = [&](int e, float2 v) {
        const int t = e / (M * 8), rem = e - t * (M * 8);
        const int row = 16 * (rb * T + t) + 2 * (rem & 7);
        if (row < N) *reinterpret_cast<__half2*>(p.y + static_cast<size_t>(rem >> 3) * N + row) = __floats2half2_rn(v.x, v.y);
    };
    if (CS > 1) cluster_wait();                       // every CTA of the cluster has started: its shared memory exists
    for (int e = tid; e < pairs; e += nthreads) {
        float2 sum = make_float2(0.f, 0.f);
        for (int k = 0; k < KW; ++k) {
            const float2 v = *reinterpret_cast<const float2*>(red + k * T * M * 16 + 2 * e);
            sum.x += v.x;
            sum.y += v.y;
        }
        if (CS == 1) {
            store_out(e, sum);
        } else {
            // hand the pair to the CTA of the cluster that owns it
            const int owner = e / share;
            st_cluster_f32x2(sbase + sm.cred + 8u * (rank * share + (e - owner * share)), owner, sum);
        }
    }
    if (CS == 1) return;

    // ---- split-K: every CTA adds, in rank order, the partials it received for its share of pairs -----
    cluster_sync_all();
    const float2* cred = reinterpret_cast<const float2*>(smem + sm.cred);
    for (int i = tid; i < share; i += nthreads) {
        const int e = rank * share + i;
        if (e < pairs) {
            float2 sum = make_float2(0.f, 0.f);
            for (int s = 0; s < CS; ++s) {
                const float2 v = cred[s * share + i];
                sum.x += v.x;
                sum.y += v.y;
            }
            store_out(e, sum);
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
struct GemvPlan {
    int NT, W, T, CS, GC;
    int region_bytes, max_groups, max_slots;
    bool two_bufs;
    bool pre;                // x pre-staged in global scratch
    uint32_t smem_bytes;
    uint16_t kbegin[kMaxCluster + 1];
};

static int device_sm_count() {
    static std::atomic<int> cached[64];       // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// k-slice boundaries at the groups where the running bit count crosses i/cs of the total.
static void split_groups(const GroupTable& gt, int cs, GemvPlan* pl) {
    const int G = gt.G;
    const int total = gt.prefix[G];
    pl->kbegin[0] = 0;
    int j = 0;
    for (int i = 1; i < cs; ++i) {
        const int target = (total * i + cs / 2) / cs;
        while (j < G && gt.prefix[j] < target) ++j;
        if (j <= pl->kbegin[i - 1]) j = pl->kbegin[i - 1] + 1;   // every slice gets at least one group
        if (j > G - (cs - i)) j = G - (cs - i);
        pl->kbegin[i] = static_cast<uint16_t>(j);
    }
    pl->kbegin[cs] = static_cast<uint16_t>(G);
    int mg = 0;
    for (int i = 0; i < cs; ++i) mg = mg > (pl->kbegin[i + 1] - pl->kbegin[i]) ? mg : (pl->kbegin[i + 1] - pl->kbegin[i]);
    pl->max_groups = mg;
    pl->CS = cs;
}

// Sizes that depend on the chunk length: the largest chunk in bytes and in slices.
static void size_chunks(const GroupTable& gt, int gc, GemvPlan* pl) {
    int ms = 0, mb = 0;
    for (int i = 0; i < pl->CS; ++i)
        for (int a = pl->kbegin[i]; a < pl->kbegin[i + 1]; a += gc) {
            const int b = a + gc < pl->kbegin[i + 1] ? a + gc : pl->kbegin[i + 1];
            int slots = 0;
            for (int q = a; q < b; ++q) slots += slice_count(gt.bits[q]);
            const int bytes = 256 * (gt.prefix[b] - gt.prefix[a]) + 64 * (b - a);
            ms = ms > slots ? ms : slots;
            mb = mb > bytes ? mb : bytes;
        }
    pl->GC = gc;
    pl->max_slots = ms;
    pl->region_bytes = mb * pl->T;
    pl->two_bufs = pl->max_groups > gc;
}

// Deterministic launch plan for (M, N, K, bit map) on the current device.  x is staged once per
// CTA, so a CTA takes as many tiles (up to 8, one per warp) as still leaves two CTAs per SM; the
// k-range is cut so that a warp sees about two groups (its instruction stream is the critical
// path) and further while the grid is smaller than two CTAs per SM; chunks
// are as long as shared memory allows while CTAs of consecutive layers can still share an SM.
// Returns false if a single group does not fit (cannot happen within the documented limits).
static bool plan_gemv(int M, int N, const GroupTable& gt, bool pre, GemvPlan* pl) {
    const int G = gt.G;
    pl->pre = pre;
    pl->NT = M <= 8 ? 1 : 2;
    pl->W = kMaxWarps;
    const int sms = device_sm_count();
    const int tiles = N / 16;
    const int cs_max = G < kMaxCluster ? G : kMaxCluster;
    int T = kMaxWarps;
    while (T > 1 && ((tiles + T - 1) / T) * cs_max < 2 * sms) T >>= 1;
    pl->T = T;
    const int rb = (tiles + T - 1) / T;
    int cs = (G * T / kMaxWarps + 1) / 2;
    if (cs < 1) cs = 1;
    if (cs > cs_max) cs = cs_max;
    while (cs < cs_max && rb * cs < 2 * sms) ++cs;
    split_groups(gt, cs, pl);
    // up to two chunks under 48 KB if possible, else the fewest chunks under 100 KB (two CTAs
    // per SM), else whatever fits
    const uint32_t budgets[3] = {48 * 1024, 100 * 1024, 220 * 1024};
    for (int bi = 0; bi < 3; ++bi)
        for (int nc = 1; nc <= (bi == 0 && pl->max_groups > 2 ? 2 : pl->max_groups); ++nc) {
            size_chunks(gt, (pl->max_groups + nc - 1) / nc, pl);
            const uint32_t need = make_smem_map(M, pl->W, pl->T, pl->CS, pl->GC, pl->region_bytes, pl->max_slots, pl->two_bufs, pl->pre).total;
            if (need > budgets[bi]) continue;
            pl->smem_bytes = need;
            return true;
        }
    return false;
}

// Scratch layout of the pre-staged mode: header, then sums [G][16] float2, then fragments.
static size_t prestage_sxe_offset() { return kWsHeader; }
static size_t prestage_xs_offset(int G) { return kWsHeader + static_cast<size_t>(G) * 128; }
static size_t prestage_bytes(int M, const GroupTable& gt) {
    int slots = gt.G;
    for (int j = 0; j < gt.G; ++j) slots += gt.bits[j] == 3 ? 1 : 0;
    return prestage_xs_offset(gt.G) + static_cast<size_t>(slots) * 8 * M * 32;
}

static cudaError_t launch_stage_x(const StageParams& sp, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>((sp.M * sp.G + 7) / 8), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_stage_x_kernel, sp);
}

template <int NT, bool PRE>
static cudaError_t launch_gemv(const GemvParams& prm, const GemvPlan& pl, cudaStream_t stream) {
    static std::atomic<bool> attr_set[64];    // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemv_kernel<NT, PRE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(pl.CS), static_cast<unsigned>((prm.N / 16 + pl.T - 1) / pl.T), 1);
    cfg.blockDim = dim3(static_cast<unsigned>(pl.W * 32), 1, 1);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(pl.CS);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemv_kernel<NT, PRE>, prm);
}

}  // namespace slim

extern "C" {

int slim_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes) {
    if (out_bytes == nullptr || M < 0) return SLIM_ERR_INVALID_ARG;
    if (slim::is_small_group(g)) return slim::small_workspace_bytes(M, N, K, g, bits_host, out_bytes);
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (M > SLIM_GEMV_MAX_M && N > 0) *out_bytes = slim::gemm_workspace_bytes(M, N, gt.G);
    else if (M >= slim::kPreStageMinM && N > 0 && K > 0) *out_bytes = slim::prestage_bytes(M, gt);
    else *out_bytes = slim::kWsHeader;
    if (M >= 1 && M <= SLIM_GEMV_MAX_M && N > 0 && K > 0) {       // large layers go through the layer-set kernels
        const size_t routed = slim::gemv_route_workspace_bytes(M, N, K, g, bits_host, gt);
        if (routed > *out_bytes) *out_bytes = routed;
    }
    return SLIM_OK;
}

int slim_gemv_plan(int M, int N, int K, int g, const uint8_t* bits_host, int* out6) {
    if (out6 == nullptr || M < 1 || M > SLIM_GEMV_MAX_M) return SLIM_ERR_INVALID_ARG;
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    if (N == 0 || K == 0) return SLIM_ERR_INVALID_ARG;
    slim::GemvPlan pl;
    if (!slim::plan_gemv(M, N, gt, M >= slim::kPreStageMinM, &pl)) return SLIM_ERR_UNSUPPORTED;
    out6[0] = pl.T; out6[1] = pl.CS; out6[2] = (N / 16 + pl.T - 1) / pl.T; out6[3] = static_cast<int>(pl.smem_bytes);
    out6[4] = pl.NT; out6[5] = pl.GC;
    return SLIM_OK;
}

int slim_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (workspace == nullptr || workspace_bytes < slim::kWsHeader) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;
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
    if (slim::is_small_group(g))
        return slim::small_linear(x, packed, bits_host, scales, zeros, y, M, N, K, g, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
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
    if (workspace == nullptr || workspace_bytes < slim::kWsHeader) return SLIM_ERR_WORKSPACE;
    if (!slim::aligned16(workspace)) return SLIM_ERR_ALIGNMENT;

    // A layer large enough to feed the persistent ring on its own goes through the layer-set kernels, if the workspace
    // has room for their plan and staged activations (slim_workspace_bytes asks for it).
    {
        const int routed = slim::gemv_route(x, packed, bits_host, gt, scales, zeros, y, M, N, K, g, workspace, workspace_bytes, s);
        if (routed <= 0) return routed;
    }
    // A single token: the integer form with the whole K of a few tiles per CTA, if the layer fits it.
    {
        const int taken = slim::gemv_one(x, packed, gt, scales, zeros, y, M, N, K, workspace, s);
        if (taken <= 0) return taken;
    }
    // From kPreStageMinM tokens on, a small kernel puts x into fragment order once, in the
    // workspace; with a workspace too small for that every CTA stages its own part of x.
    const bool pre = M >= slim::kPreStageMinM && workspace_bytes >= slim::prestage_bytes(M, gt);
    slim::GemvPlan pl;
    if (!slim::plan_gemv(M, N, gt, pre, &pl)) return SLIM_ERR_UNSUPPORTED;

    slim::GemvParams prm;
    memset(&prm, 0, sizeof prm);
    prm.x = static_cast<const __half*>(x);
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.zeros = static_cast<const __half*>(zeros);
    prm.y = static_cast<__half*>(y);
    prm.M = M; prm.N = N; prm.K = K;
    prm.CS = pl.CS;
    prm.W = pl.W;
    prm.T = pl.T;
    prm.GC = pl.GC;
    prm.region_bytes = pl.region_bytes;
    prm.max_slots = pl.max_slots;
    prm.two_bufs = pl.two_bufs ? 1 : 0;
    memcpy(prm.kbegin, pl.kbegin, sizeof prm.kbegin);
    prm.pre3[0] = 0;
    for (int j = 0; j < SLIM_MAX_GROUPS; ++j)
        prm.pre3[j + 1] = static_cast<uint16_t>(prm.pre3[j] + (j < gt.G && gt.bits[j] == 3 ? 1 : 0));
    prm.gt = gt;

    cudaError_t e;
    if (pre) {
        uint8_t* ws = static_cast<uint8_t*>(workspace);
        slim::StageParams sp;
        memset(&sp, 0, sizeof sp);
        sp.x = prm.x;
        sp.sxe_g = reinterpret_cast<float2*>(ws + slim::prestage_sxe_offset());
        sp.xs_g = ws + slim::prestage_xs_offset(gt.G);
        sp.M = M; sp.K = K; sp.G = gt.G;
        memcpy(sp.pre3, prm.pre3, sizeof sp.pre3);
        memcpy(sp.bits, gt.bits, sizeof sp.bits);
        prm.xs_g = sp.xs_g;
        prm.sxe_g = sp.sxe_g;
        SLIM_CUDA_TRY(slim::launch_stage_x(sp, s));
        e = pl.NT == 1 ? slim::launch_gemv<1, true>(prm, pl, s) : slim::launch_gemv<2, true>(prm, pl, s);
    } else {
        e = pl.NT == 1 ? slim::launch_gemv<1, false>(prm, pl, s) : slim::launch_gemv<2, false>(prm, pl, s);
    }
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

}  // extern "C"
