// One layer, one token, one launch: the inference kernel of App. B.2 in its own launch mode (a kernel per linear
// layer), in the integer form of the single-token layer sets (slim_gemv_i8.cuh).
//
// A decode-sized layer is a few megabytes, so the launch is over in a few microseconds and what counts is the
// length of the dependent chain inside a CTA, not the instruction count.  Hence:
//
//  * a CTA owns 2, 4, 6 or 8 tiles of 16 rows and the WHOLE K: no partial sums leave the CTA and there is no second
//    pass.  The tile count is the smallest for which all CTAs of the layer are resident at once (else the one that
//    needs the fewest waves).
//  * warp w owns the groups w, w + 16, ... of the CTA's tiles: it brings their slices with one cp.async.bulk per
//    group onto a barrier of its own, their scales and zeros with 16-byte cp.async, multiplies and folds.  Warps
//    meet at the end to add their sixteen partial sums per row in warp order (deterministic).
//  * the digit form of x is the same for every CTA and costs a warp about as much as a group's products, so the
//    CTAs of a cluster of eight share it: CTA r stages the groups r, r + 8, ... (one per warp) and writes each
//    record into the shared memory of all eight through distributed shared memory; one cluster barrier follows.
//  * everything that does not depend on x (the slices, scales, zeros) is requested BEFORE griddepcontrol.wait, and
//    the dependents are released right after, so with programmatic dependent launch the loads of layer l + 1 are in
//    flight while layer l computes.
//  * a set of a few single-token layers (q/k/v, gate/up) whose CTAs are all resident at once is ONE launch of the
//    same body: every layer owns whole clusters, a CTA reads its layer's descriptor from the plan buffer first.
//
// Every wait on a barrier in memory is bounded and reports through the workspace status word.
#include "slim_common.cuh"
#include "slim_gemv_i8.cuh"

#include <atomic>
#include <cstring>
#include <vector>

namespace slim {

constexpr int kOneWarps = 16;
constexpr int kOneThreads = 32 * kOneWarps;
constexpr int kOneCluster = 8;                          // CTAs that share the staging of x (4 where eight do not all fit)
constexpr int kOneMaxPairs = 4;                         // tile pairs per CTA
constexpr uint32_t kOneOffAbort = 8 * kOneWarps;        // after the warps' barriers
constexpr uint32_t kOneOffXs = 256;                     // per warp: 128 ints of scratch for the digit staging, later its partial sums
constexpr uint32_t kOneOffDesc = kOneOffXs + kOneWarps * 512;   // the layer's descriptor, when it comes from the plan buffer of a set
constexpr uint32_t kOneOffS = kOneOffDesc + 1408;

struct OneParams {
    const __half* x;
    const uint8_t* packed;
    const __half* scales;
    const __half* zeros;
    __half* y;
    uint8_t* ws;                            // status word at offset 0 (single-layer launch; a set passes it to the kernel)
    int N, G, gshift;
    int one;                                // 1: a multiplier the compiler cannot fold (selects done as integer multiply-adds)
    uint32_t off_z, off_x, off_w;           // shared-memory offsets: zeros, activation records, slices (scales at kOneOffS)
    uint16_t prefix[SLIM_MAX_GROUPS + 1];   // bits before K-tile j
    uint16_t pre3[SLIM_MAX_GROUPS + 1];     // 3-bit K-tiles before j (their activation records hold two slices)
    uint8_t bits[SLIM_MAX_GROUPS];
};
static_assert(sizeof(OneParams) % 16 == 0 && sizeof(OneParams) <= kOneOffS - kOneOffDesc, "descriptors are copied in 16-byte pieces");

__device__ __forceinline__ void st_cluster_u32x4(uint32_t local_addr, uint32_t rank, uint4 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(remote), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// One K-tile of B bits for the PAIRS tile pairs of the CTA: integer MMAs on byte-masked words, then the fold
// acc += s (D 2^(-S-Pc) - z sum_x) per (row, K-tile); lane pair c >> 1 folds tile c >> 1 of every pair.
template <int B, int PAIRS>
__device__ __forceinline__ void one_group(const OneParams& p, uint32_t wj, uint32_t rec, uint32_t sj, uint32_t zj, int lane,
                                          float (&acc)[PAIRS][2]) {
    const int gq = lane >> 2, c = lane & 3;
    const int tsel = c >> 1;
    const int m0 = tsel ? 0 : p.one, m1 = tsel ? p.one : 0;
    const float ma = (c & 1) ? 256.f : 16777216.f, mb = (c & 1) ? 1.f : 65536.f;
    constexpr int kMagicBits = 0x4B400000;                 // 1.5 * 2^23: adding an integer |v| < 2^22 to these bits gives the float 12582912 + v
    constexpr float kMagic = 12582912.f;
    const uint2 tkw = lds64(rec);
    const float sum_x = __uint_as_float(tkw.x), e = __uint_as_float(tkw.y);
    const float ka = ma * e, kb = mb * e;
    const uint32_t xs_lane = rec + 128 + ((gq & 3) * 4 + c) * 8;
#pragma unroll
    for (int tp = 0; tp < PAIRS; ++tp) {
        const uint32_t item0 = wj + 8u * lane + static_cast<uint32_t>(2 * tp) * (256u * B);
        int di[2][2][4];
        auto run_pass = [&](auto wtag, auto first_tag, int unit0, uint32_t xs) {
            constexpr int WD = decltype(wtag)::value;
            constexpr bool FIRST = decltype(first_tag)::value != 0;
            constexpr uint32_t kByteMask = 0x01010101u * ((1u << WD) - 1u);
            constexpr int NW = WD;
            uint2 wd[2][NW];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const uint32_t item = item0 + t * (256u * B) + 256u * unit0;
#pragma unroll
                for (int u = 0; u < NW; ++u) wd[t][u] = lds64(item + 256u * u);
            }
#pragma unroll
            for (int mi = 0; mi < 4; ++mi) {
                const uint2 bv = lds64(xs + mi * 128);
                const int w_lo = WD == 4 ? 2 * (mi >> 1) : 0, w_hi = WD == 1 ? 0 : w_lo + 1;
                const int pos_lo = i8_pos(WD, mi, 0), pos_hi = i8_pos(WD, mi, 1);
                const uint32_t m_lo = kByteMask << (WD * pos_lo), m_hi = kByteMask << (WD * pos_hi);
                const bool top_lo = WD * (pos_lo + 1) == 8, top_hi = WD * (pos_hi + 1) == 8;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const uint32_t a0 = top_lo ? wd[t][w_lo].x : wd[t][w_lo].x & m_lo, a1 = top_lo ? wd[t][w_lo].y : wd[t][w_lo].y & m_lo;
                    const uint32_t a2 = top_hi ? wd[t][w_hi].x : wd[t][w_hi].x & m_hi, a3 = top_hi ? wd[t][w_hi].y : wd[t][w_hi].y & m_hi;
                    if (FIRST && mi < 2) mma_i8_first(di[t][mi & 1], a0, a1, a2, a3, bv);
                    else mma_i8(di[t][mi & 1], a0, a1, a2, a3, bv);
                }
            }
        };
        if (B == 1) run_pass(WidthTag<1>{}, WidthTag<1>{}, 0, xs_lane);
        if (B == 2) run_pass(WidthTag<2>{}, WidthTag<1>{}, 0, xs_lane);
        if (B == 3) { run_pass(WidthTag<2>{}, WidthTag<1>{}, 0, xs_lane); run_pass(WidthTag<1>{}, WidthTag<0>{}, 2, xs_lane + 512); }
        if (B == 4) run_pass(WidthTag<4>{}, WidthTag<1>{}, 0, xs_lane);
        const uint32_t sz_lane = static_cast<uint32_t>((2 * tp + tsel) * 32 + gq * 4);
        const uint32_t s2 = lds32(sj + sz_lane);
        const uint32_t z2 = lds32(zj + sz_lane);
        float f[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            int v = kMagicBits;
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) v += di[0][ch][r] * m0 + di[1][ch][r] * m1;
            f[r] = __int_as_float(v) - kMagic;                        // exact
        }
        const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
        const float2 zf = __half22float2(*reinterpret_cast<const __half2*>(&z2));
        float r0 = fmaf(f[0], ka, f[1] * kb);
        float r1 = fmaf(f[2], ka, f[3] * kb);
        r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
        r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
        acc[tp][0] = fmaf(sf.x, fmaf(-zf.x, sum_x, r0), acc[tp][0]);
        acc[tp][1] = fmaf(sf.y, fmaf(-zf.y, sum_x, r1), acc[tp][1]);
    }
}

// The work of CTA `bid` of layer p (see the head of the file).
template <int PAIRS>
__device__ __forceinline__ void one_body(const OneParams& p, int bid, uint8_t* status, uint8_t* smem) {
    constexpr int TPC = 2 * PAIRS;                         // tiles per CTA
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort = reinterpret_cast<volatile int*>(smem + kOneOffAbort);
    const uint32_t bar = sbase + 8u * warp;
    const int tile0 = TPC * bid;
    const int tiles_here = max(min(TPC, (p.N >> 4) - tile0), 0);  // 0: a CTA that only fills up its cluster
    const int ng = (p.G - warp + kOneWarps - 1) / kOneWarps;      // this warp's K-tiles: warp, warp + 16, ...
    const uint32_t rank = cluster_ctarank();
    uint32_t nrank;                                        // CTAs of the cluster: 8 or 4
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(nrank));

    // ---- requests that do not depend on x
    if (lane == 0) {
        sb::init(bar, 1);
        if (warp == 0) *abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();                                       // the abort flag is clear before any warp can poll it
    {
        const int j = warp + kOneWarps * lane;             // lane i brings the slices of the warp's i-th K-tile
        const uint32_t b = lane < ng ? p.bits[j] : 0u;
        const uint32_t bytes = static_cast<uint32_t>(tiles_here) * 256u * b;
        const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
        if (lane == 0) sb::expect_tx(bar, total);
        __syncwarp();
        if (lane < ng && bytes != 0)
            sb::bulk_g2s(sbase + p.off_w + static_cast<uint32_t>(TPC) * 256u * p.prefix[j],
                         p.packed + 16ull * p.N * p.prefix[j] + static_cast<size_t>(tile0) * 256 * b, bytes, bar);
        // scales and zeros of the warp's K-tiles, 16 bytes (8 rows) at a time
        const int chunks = 2 * tiles_here;
        for (int i = lane; i < ng * chunks * 2; i += 32) {
            const int which = i & 1, q = i >> 1, gi = q / chunks, ch = q - gi * chunks;
            const int jj = warp + kOneWarps * gi;
            const __half* src = (which ? p.zeros : p.scales) + static_cast<size_t>(jj >> p.gshift) * p.N + 16 * tile0 + 8 * ch;
            cp_async16(sbase + (which ? p.off_z : kOneOffS) + static_cast<uint32_t>(jj) * (32u * TPC) + 16u * ch, src);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    pdl_launch_dependents();
    pdl_wait();                                            // x may be the output of the kernel before

    // ---- the activations as digits: this CTA's share of the K-tiles, written into every CTA of the cluster
    int* Xs = reinterpret_cast<int*>(smem + kOneOffXs + 512 * warp);
    for (int j = static_cast<int>(rank + nrank * warp); j < p.G; j += static_cast<int>(nrank) * kOneWarps) {
        const uint32_t off = p.off_x + static_cast<uint32_t>(staged_group_offset(j, p.pre3[j], 2));
        stage_group_i8(p.x + SLIM_GROUP * j, smem + off, p.bits[j], lane, Xs);
        __syncwarp();
        const int pieces = (128 + 512 * slice_count(p.bits[j])) / 16;
        for (int i = lane; i < pieces; i += 32) {
            const uint4 v = lds128(sbase + off + 16u * i);
            for (uint32_t r = 0; r < nrank; ++r)
                if (r != rank) st_cluster_u32x4(sbase + off + 16u * i, r, v);
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");

    float acc[PAIRS][2];
#pragma unroll
    for (int tp = 0; tp < PAIRS; ++tp) acc[tp][0] = acc[tp][1] = 0.f;
    const bool ok = __all_sync(0xffffffffu, sb::wait(bar, 0, abort));
    if (ok && tiles_here > 0) {
        for (int gi = 0; gi < ng; ++gi) {
            const int j = warp + kOneWarps * gi;
            const uint32_t wj = sbase + p.off_w + static_cast<uint32_t>(TPC) * 256u * p.prefix[j];
            const uint32_t rec = sbase + p.off_x + static_cast<uint32_t>(staged_group_offset(j, p.pre3[j], 2));
            const uint32_t sj = sbase + kOneOffS + static_cast<uint32_t>(j) * (32u * TPC);
            const uint32_t zj = sbase + p.off_z + static_cast<uint32_t>(j) * (32u * TPC);
            switch (p.bits[j]) {
                case 1: one_group<1, PAIRS>(p, wj, rec, sj, zj, lane, acc); break;
                case 2: one_group<2, PAIRS>(p, wj, rec, sj, zj, lane, acc); break;
                case 3: one_group<3, PAIRS>(p, wj, rec, sj, zj, lane, acc); break;
                default: one_group<4, PAIRS>(p, wj, rec, sj, zj, lane, acc); break;
            }
        }
    }
    // ---- the warps' partial sums, added in warp order
    __syncwarp();
    float* mine = reinterpret_cast<float*>(smem + kOneOffXs + 512 * warp);      // [TPC * 16] floats, the scratch is free now
    {
        const int gq = lane >> 2, c = lane & 3;
        if ((c & 1) == 0) {
#pragma unroll
            for (int tp = 0; tp < PAIRS; ++tp)
                *reinterpret_cast<float2*>(mine + (2 * tp + (c >> 1)) * 16 + 2 * gq) = make_float2(acc[tp][0], acc[tp][1]);
        }
    }
    __syncthreads();
    if (*abort != 0) {
        if (tid == 0) atomicOr(reinterpret_cast<unsigned int*>(status), 1u);
        return;
    }
    if (tid < 8 * tiles_here) {                            // a pair of rows per thread
        const float* all = reinterpret_cast<const float*>(smem + kOneOffXs);
        float2 sum = *reinterpret_cast<const float2*>(all + 2 * tid);
#pragma unroll
        for (int w = 1; w < kOneWarps; ++w) {
            const float2 v = *reinterpret_cast<const float2*>(all + 128 * w + 2 * tid);
            sum.x += v.x;
            sum.y += v.y;
        }
        *reinterpret_cast<__half2*>(p.y + 16 * tile0 + 2 * tid) = __floats2half2_rn(sum.x, sum.y);
    }
}

template <int PAIRS>
__global__ void __launch_bounds__(kOneThreads, PAIRS == 1 ? 2 : 1) gemv_one_kernel(const __grid_constant__ OneParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    one_body<PAIRS>(p, static_cast<int>(blockIdx.x), p.ws, smem);
}

// Several layers in one launch, every CTA resident at once: layer l owns the CTAs cta0[l] .. cta0[l + 1] (whole
// clusters).  The descriptors live in the plan buffer of the set; a CTA copies its own into shared memory first.
template <int PAIRS>
__global__ void __launch_bounds__(kOneThreads, PAIRS == 1 ? 2 : 1) gemv_one_set_kernel(const OneParams* __restrict__ layers,
                                                                                     const int* __restrict__ cta0, int n_layers,
                                                                                     uint8_t* status) {
    extern __shared__ __align__(128) uint8_t smem[];
    int l = 0;
    while (l + 1 < n_layers && cta0[l + 1] <= static_cast<int>(blockIdx.x)) ++l;
    const uint4* src = reinterpret_cast<const uint4*>(layers + l);
    uint4* dst = reinterpret_cast<uint4*>(smem + kOneOffDesc);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(OneParams) / 16); i += kOneThreads) dst[i] = src[i];
    __syncthreads();
    one_body<PAIRS>(*reinterpret_cast<const OneParams*>(smem + kOneOffDesc), static_cast<int>(blockIdx.x) - cta0[l], status, smem);
}

template <int PAIRS>
static cudaError_t launch_one(const OneParams& prm, int grid, int cluster, size_t smem, cudaStream_t stream) {
    static std::atomic<bool> attr_set[64];    // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemv_one_kernel<PAIRS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kOneThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemv_one_kernel<PAIRS>, prm);
}

// Clusters of the kernel that can be resident at once with `smem` bytes of dynamic shared memory (0 on failure).
template <int PAIRS>
static int one_max_clusters(size_t smem, int cluster) {
    if (cudaFuncSetAttribute(gemv_one_kernel<PAIRS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(cluster), 1, 1);
    cfg.blockDim = dim3(kOneThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemv_one_kernel<PAIRS>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

// The same, asked once per device for the two sizes that matter: a CTA small enough for two per SM, and the largest.
constexpr size_t kOneHalfSm = 112 * 1024;
static int one_clusters_cached(int pairs, size_t smem, int cluster) {
    static std::atomic<int> cache[64][kOneMaxPairs][2][2];  // 0: not asked yet; idempotent, so a race repeats the query
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const int cls = smem <= kOneHalfSm ? 0 : 1, ci = cluster == kOneCluster ? 0 : 1;
    int v = cache[dev][pairs - 1][cls][ci].load();
    if (v == 0) {
        const size_t ask = cls == 0 ? kOneHalfSm : 224 * 1024;
        v = pairs == 1 ? one_max_clusters<1>(ask, cluster) : pairs == 2 ? one_max_clusters<2>(ask, cluster)
          : pairs == 3 ? one_max_clusters<3>(ask, cluster) : one_max_clusters<4>(ask, cluster);
        cache[dev][pairs - 1][cls][ci].store(v > 0 ? v : -1);
    }
    return v > 0 ? v : 0;
}

// Shared-memory layout of a CTA with `pairs` tile pairs of a layer; false if it does not fit.
struct OneShape {
    size_t smem;
    uint32_t off_z, off_x, off_w;
};
static bool one_shape(const GroupTable& gt, int pairs, OneShape* o) {
    int n3 = 0;
    for (int j = 0; j < gt.G; ++j) n3 += gt.bits[j] == 3 ? 1 : 0;
    const size_t x_bytes = staged_group_offset(gt.G, n3, 2);
    const int tpc = 2 * pairs;
    const size_t sz = static_cast<size_t>(gt.G) * 32 * tpc;
    const size_t oz = kOneOffS + sz, ox = (oz + sz + 127) / 128 * 128, ow = (ox + x_bytes + 127) / 128 * 128;
    o->smem = ow + static_cast<size_t>(tpc) * 256 * gt.prefix[gt.G];
    o->off_z = static_cast<uint32_t>(oz); o->off_x = static_cast<uint32_t>(ox); o->off_w = static_cast<uint32_t>(ow);
    return o->smem <= 224 * 1024;
}
static void one_fill(OneParams* out, const void* x, const void* packed, const void* scales, const void* zeros, void* y, void* workspace,
                     int N, const GroupTable& gt, const OneShape& sh) {
    OneParams& prm = *out;
    memset(&prm, 0, sizeof prm);
    prm.x = static_cast<const __half*>(x);
    prm.packed = static_cast<const uint8_t*>(packed);
    prm.scales = static_cast<const __half*>(scales);
    prm.zeros = static_cast<const __half*>(zeros);
    prm.y = static_cast<__half*>(y);
    prm.ws = static_cast<uint8_t*>(workspace);
    prm.N = N; prm.G = gt.G; prm.gshift = gt.gshift;
    prm.one = 1;
    prm.off_z = sh.off_z; prm.off_x = sh.off_x; prm.off_w = sh.off_w;
    memcpy(prm.prefix, gt.prefix, sizeof prm.prefix);
    memcpy(prm.bits, gt.bits, sizeof prm.bits);
    prm.pre3[0] = 0;
    for (int j = 0; j < SLIM_MAX_GROUPS; ++j)
        prm.pre3[j + 1] = static_cast<uint16_t>(prm.pre3[j] + (j < gt.G && gt.bits[j] == 3 ? 1 : 0));
}
static int pad_to(int v, int m) { return (v + m - 1) / m * m; }

// Enqueues the layer on the single-token kernel and returns SLIM_OK, a negative status on failure, or 1 if this shape
// does not fit it (the caller then takes the general kernel): the whole K of a CTA's tiles, their scales and zeros and
// the digit form of x must fit the shared memory of a CTA.  Among the tile counts that fit, the one that needs the
// fewest waves of resident CTAs is taken (one wave for the decode shapes of 7B and 13B models), the smallest of equals.
int gemv_one(const void* x, const void* packed, const GroupTable& gt, const void* scales, const void* zeros, void* y,
             int M, int N, int K, void* workspace, cudaStream_t stream) {
    (void)K;
    if (M != 1 || N <= 0 || gt.G < 1) return 1;
    const int tiles = N >> 4;
    int pairs = 0, cluster = 0, best_waves = 1 << 30;
    OneShape shape;
    for (int pr = 1; pr <= kOneMaxPairs; ++pr) {
        OneShape sh;
        if (!one_shape(gt, pr, &sh)) break;
        for (int cs = kOneCluster; cs >= 4; cs /= 2) {                         // eight CTAs share the staging, or four
            const int grid = pad_to((tiles + 2 * pr - 1) / (2 * pr), cs), resident = one_clusters_cached(pr, sh.smem, cs) * cs;
            if (resident <= 0) continue;
            const int waves = (grid + resident - 1) / resident;
            if (waves < best_waves) { best_waves = waves; pairs = pr; cluster = cs; shape = sh; }
        }
        if (best_waves == 1) break;
    }
    if (pairs == 0) return 1;
    OneParams prm;
    one_fill(&prm, x, packed, scales, zeros, y, workspace, N, gt, shape);
    const int grid = pad_to((tiles + 2 * pairs - 1) / (2 * pairs), cluster);
    const cudaError_t e = pairs == 1 ? launch_one<1>(prm, grid, cluster, shape.smem, stream)
                        : pairs == 2 ? launch_one<2>(prm, grid, cluster, shape.smem, stream)
                        : pairs == 3 ? launch_one<3>(prm, grid, cluster, shape.smem, stream)
                                     : launch_one<4>(prm, grid, cluster, shape.smem, stream);
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

// ------------------------------------------------------------------------------------------ small single-token sets, resident
// A set of single-token layers whose CTAs are all resident at once (q/k/v, gate/up: a few layers) runs as ONE launch of
// the kernel above instead of the staging kernel plus the persistent ring: no ring to fill and drain, no second kernel.
constexpr int kOneSetMaxLayers = 64;

template <int PAIRS>
static cudaError_t launch_one_set(const OneSetPlan& pl, const void* plan, int n_layers, void* workspace, cudaStream_t stream) {
    static std::atomic<bool> attr_set[64];    // zero-initialised; set-up is idempotent, so a race repeats it harmlessly
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemv_one_set_kernel<PAIRS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(pl.grid), 1, 1);
    cfg.blockDim = dim3(kOneThreads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(pl.cluster);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const uint8_t* base = static_cast<const uint8_t*>(plan);
    return cudaLaunchKernelEx(&cfg, gemv_one_set_kernel<PAIRS>, reinterpret_cast<const OneParams*>(base + kOneSetPlanHeader),
                              reinterpret_cast<const int*>(base), n_layers, static_cast<uint8_t*>(workspace));
}

int one_set_plan(const slim_layer* layers, int n_layers, int g, void* plan, size_t plan_bytes, cudaStream_t stream, OneSetPlan* out) {
    if (n_layers < 1 || n_layers > kOneSetMaxLayers || g < SLIM_GROUP) return 1;
    if (plan_bytes < kOneSetPlanHeader + static_cast<size_t>(n_layers) * sizeof(OneParams)) return 1;
    std::vector<GroupTable> gt(static_cast<size_t>(n_layers));
    for (int l = 0; l < n_layers; ++l) {
        if (layers[l].M != 1) return 1;
        const int st = make_group_table(layers[l].N, layers[l].K, g, layers[l].bits_host, &gt[l]);
        if (st != SLIM_OK) return st;
    }
    // one wave of resident CTAs; a set of at most four layers may take two (it is still ahead of filling and draining a ring)
    // (then with the largest tile count that fits, which needs the fewest CTAs)
    for (int waves = 1; waves <= (n_layers <= 4 ? 2 : 1); ++waves)
    for (int step = 1; step <= kOneMaxPairs; ++step) {
        const int pr = waves == 1 ? step : kOneMaxPairs + 1 - step;
        OneShape sh[kOneSetMaxLayers];
        size_t smem = 0;
        bool fits = true;
        for (int l = 0; l < n_layers && fits; ++l) {
            fits = one_shape(gt[l], pr, &sh[l]);
            smem = smem > sh[l].smem ? smem : sh[l].smem;
        }
        if (!fits) { if (waves == 1) break; else continue; }
        for (int cs = kOneCluster; cs >= 4; cs /= 2) {
            int cta0[kOneSetMaxLayers + 1];
            cta0[0] = 0;
            for (int l = 0; l < n_layers; ++l) cta0[l + 1] = cta0[l] + pad_to(((layers[l].N >> 4) + 2 * pr - 1) / (2 * pr), cs);
            if (cta0[n_layers] > waves * one_clusters_cached(pr, smem, cs) * cs) continue;
            // taken: descriptors and CTA ranges into the plan buffer (pageable sources are staged before the copies return)
            std::vector<OneParams> prm(static_cast<size_t>(n_layers));
            for (int l = 0; l < n_layers; ++l)
                one_fill(&prm[l], layers[l].x, layers[l].packed, layers[l].scales, layers[l].zeros, layers[l].y, nullptr, layers[l].N, gt[l], sh[l]);
            uint8_t* base = static_cast<uint8_t*>(plan);
            SLIM_CUDA_TRY(cudaMemcpyAsync(base, cta0, static_cast<size_t>(n_layers + 1) * sizeof(int), cudaMemcpyHostToDevice, stream));
            SLIM_CUDA_TRY(cudaMemcpyAsync(base + kOneSetPlanHeader, prm.data(), static_cast<size_t>(n_layers) * sizeof(OneParams), cudaMemcpyHostToDevice, stream));
            out->pairs = pr; out->cluster = cs; out->grid = cta0[n_layers]; out->smem = smem;
            return SLIM_OK;
        }
    }
    return 1;
}

int one_set_launch(const OneSetPlan& pl, const void* plan, int n_layers, void* workspace, cudaStream_t stream) {
    if (pl.pairs < 1 || pl.pairs > kOneMaxPairs || (pl.cluster != 4 && pl.cluster != kOneCluster) || pl.grid < pl.cluster ||
        pl.grid % pl.cluster != 0 || pl.smem > 224 * 1024 || n_layers < 1 || n_layers > kOneSetMaxLayers)
        return SLIM_ERR_INVALID_ARG;
    const cudaError_t e = pl.pairs == 1 ? launch_one_set<1>(pl, plan, n_layers, workspace, stream)
                        : pl.pairs == 2 ? launch_one_set<2>(pl, plan, n_layers, workspace, stream)
                        : pl.pairs == 3 ? launch_one_set<3>(pl, plan, n_layers, workspace, stream)
                                        : launch_one_set<4>(pl, plan, n_layers, workspace, stream);
    SLIM_CUDA_TRY(e);
    return SLIM_OK;
}

}  // namespace slim
