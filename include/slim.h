/* slim.h -- C ABI of the B200 (sm_100a) group-wise mixed-precision weight-only linear layer.
 *
 * The layer is y = x * W^T with W stored quantised: the input dimension K is cut into groups of
 * g consecutive columns, 128 in the paper's main results (Algorithm 1 of the SliM-LLM paper slices w[:, b:b+beta]); group j
 * carries one bit-width b_j in {1,2,3,4} (Salience-Determined Bit Allocation, Sec. 3.2.2) and every
 * (row, group) pair carries an fp16 scale s and an fp16 zero point z.  A stored code q dequantises
 * as w = s * (q - z) (inverse of Eq. 1, written out inside Eq. 5).
 *
 * Conventions
 *   N = output features (rows of W), K = input features (columns of W), M = tokens (rows of x),
 *   G = K / g groups.  All matrices are dense row-major:
 *     x       fp16  [M][K]        device
 *     y       fp16  [M][N]        device
 *     scales  fp16  [G][N]        device   (N contiguous)
 *     zeros   fp16  [G][N]        device   (any fp16 value; integers for Eq. 1, 0.5 for Eq. 2)
 *     codes   uint8 [N][K]        device   (unpacked codes, code < 2^b_j)
 *     bits    uint8 [G]           HOST     (read during the call; values 1..4; G = K / g)
 *     packed  bytes               device   (format below, slim_packed_bytes() bytes)
 *   "device" pointers must be 16-byte aligned and are owned by the caller, who keeps them alive
 *   until the work enqueued on `stream` has finished.  No function allocates device memory,
 *   none synchronises unless it says so, and all work is enqueued on `stream` (a cudaStream_t
 *   passed as void*; NULL is the legacy default stream).  Calls never throw; they return a status.
 *
 * Threads: the entry points may be called from several host threads.  The per-device set-up that the first launch of a
 * kernel performs (a function attribute, a device query) is idempotent and published through atomics, so two threads
 * that make their first calls together repeat it harmlessly.  Calls that share a workspace, or the built-in scratch
 * of slim_mpq_gemm_static, must still be ordered on one stream.
 *
 * Limits: g in {32, 64, 128, 256, 512} (the group sizes of the paper's group-size ablation; bits, scales and zeros
 * have K / g entries or rows); K a multiple of g and of 128 with at most 256 tiles of 128 columns (1024 groups for
 * g < 128); N a multiple of 16; N = 0 or M = 0 is a successful no-op.  Anything else returns an error status and
 * enqueues nothing.  Pack, dequant, both linear entry points, the group salience and the quantizers
 * (slim_quantize_minmax, _groups, _sign1, _sqc; these also take a K that is any multiple of g), the SBA search and
 * the GPTQ loop take every g; the layer-set launch and slim_mpq_gemm_static take 128, 256 and 512
 * (SLIM_ERR_UNSUPPORTED otherwise).  Groups of 256 and 512 columns run on the tensor-core kernels of the 128-column tiles (a group is 2 or 4
 * tiles that share a row of scales and zeros); groups of 32 and 64 columns run on plain CUDA-core kernels, and the
 * batched entry point then wants room for the fp16 weights in its workspace (slim_workspace_bytes says how much).
 *
 * Packed format ("sliced bit planes", version SLIM_FORMAT_VERSION).  K is cut into K-tiles of T = min(g, 128)
 * columns; a group of more than 128 columns is g/128 consecutive K-tiles of its bit-width.  K-tiles are stored back
 * to back without padding, as the paper's deployment format does (App. B.2), so the buffer holds exactly
 * N*K*avg_bits/8 bytes.  With B_j = bits of the K-tiles before tile j:
 *   - K-tile j starts at byte (T/8)*N*B_j and holds, for each tile t of 16 consecutive rows, b_j
 *     units of 2T bytes (tile t at offset t*2T*b_j inside the K-tile);
 *   - a b-bit code is cut into slices (lo, w): b=1 -> (0,1); b=2 -> (0,2); b=3 -> (0,2),(2,1);
 *     b=4 -> (0,4); slice value = (q >> lo) & (2^w - 1).  A slice of width w owns w consecutive
 *     units, slices in the order listed;
 *   - a unit is 32 lanes x T/16 bytes.  Lane L = 4*gq + c (gq = 0..7, c = 0..3) holds two
 *     little-endian items of T/4 bits: item 0 belongs to row 16t + 2gq, item 1 to row 16t + 2gq + 1;
 *   - the item of (row r, slice (lo,w), unit u of that slice, c) has (T/4)/w fields of w bits; field f
 *     (bits [w*f, w*f + w)) stores the slice of q[r][T*j + (T/4)*c + ((T/4)/w)*u + f].
 * For g >= 128 a unit is 256 bytes and an item a 32-bit word.
 */
#ifndef SLIM_H_
#define SLIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLIM_FORMAT_VERSION 2
#define SLIM_GROUP 128           /* the paper's default group size, and the widest K-tile of the packed format */
#define SLIM_MAX_GROUPS 256      /* most K-tiles of 128 columns in a layer (K <= 32768) */
#define SLIM_GEMV_MAX_M 16
#define SLIM_GEMV_SET_MAX_M 64   /* tokens of a layer in a layer set */

enum {
    SLIM_OK = 0,
    SLIM_ERR_INVALID_ARG = -1, /* null pointer, negative size, bit-width outside 1..4, M out of range */
    SLIM_ERR_UNSUPPORTED = -2, /* group size not served by this entry point, K % g or K % 128 != 0, N % 16 != 0, too many groups */
    SLIM_ERR_ALIGNMENT = -3,   /* a device pointer is not 16-byte aligned */
    SLIM_ERR_WORKSPACE = -4,   /* workspace missing or smaller than slim_workspace_bytes() */
    SLIM_ERR_CUDA = -5,        /* a CUDA runtime call failed; see slim_last_cuda_error() */
    SLIM_ERR_TIMEOUT = -6,     /* a device-side wait gave up (reported by slim_workspace_status) */
    SLIM_ERR_STATIC_SCRATCH = -7 /* slim_mpq_gemm_static: the shape needs more than the built-in scratch */
};

/* Library / format version: (SLIM_FORMAT_VERSION << 16) | build number. */
int slim_version(void);
/* Static, NUL-terminated description of a status code. */
const char* slim_status_string(int status);
/* cudaError_t value of the most recent failing CUDA call made by this library on the calling
 * thread's process (0 if none). */
int slim_last_cuda_error(void);

/* Size of the packed buffer, N*K*avg_bits/8 bytes ("no additional padding", App. B.2). */
int slim_packed_bytes(int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes);

/* Scratch size for slim_mpq_gemv / slim_mpq_gemm with these shapes on the current device.
 * Always at least 256 (one status word).  slim_mpq_gemv needs no more up to three tokens; from
 * four tokens on it asks for room to put x into tensor-core fragment order once (a few bytes
 * per element of x) and, given less, lets every thread block do that for itself.  slim_mpq_gemm asks for
 * flags and fp32 partial tiles (128 KB per SM) when it would split tiles across CTAs (stream-K:
 * shapes whose tile count leaves the last wave of CTAs mostly idle); given a smaller workspace
 * (at least 256 bytes) it falls back to whole tiles per CTA and uses no scratch. */
int slim_workspace_bytes(int M, int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes);

/* Zeroes a workspace (status word, stream-K flags).  Must be enqueued once after allocating a
 * workspace, before its first use; the kernels leave the flags zeroed.  Calls that share a
 * workspace must be ordered on one stream. */
int slim_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream`, reads and clears the workspace status word.  Returns SLIM_OK, or
 * SLIM_ERR_TIMEOUT if a kernel using this workspace abandoned a bounded wait (its output is
 * then undefined), or SLIM_ERR_CUDA.  A kernel that gave up may have left its flags and partial sums
 * behind: after SLIM_ERR_TIMEOUT pass the workspace through slim_workspace_init before the next call
 * that uses more than its status word (slim_mpq_gemm on a shape it cuts across CTAs). */
int slim_workspace_status(void* workspace, void* stream);

/* Self-test of the device-side time-out path.  (No counterpart in the paper: it exercises the status-word
 * contract of this header.)  Enqueues one warp that waits, with the bounded wait the persistent kernels use, on a
 * barrier that nothing ever signals; after limit_us microseconds (1 .. 100000) the wait gives up, the kernel sets
 * the workspace status word the way a real time-out does, and returns by itself.  slim_workspace_status on that
 * workspace then reports SLIM_ERR_TIMEOUT once and clears the word; the workspace stays usable.  `workspace` at
 * least 256 bytes, 16-byte aligned. */
int slim_selftest_wait_timeout(void* workspace, size_t workspace_bytes, unsigned int limit_us, void* stream);

/* Packs unpacked codes into the format above (the storage step of App. B.2: "packs the weights
 * ... into integer-compressed representations based on the precision of different groups").
 * Integer work, deterministic; codes with bits above b_j set are masked to b_j bits. */
int slim_pack_weights(const uint8_t* codes, const uint8_t* bits_host, void* packed,
                      int N, int K, int g, void* stream);

/* Materialises W-hat as fp16 [N][K]:  W[n][k] = fp16_rn( f32(s) * ( f32(q) - f32(z) ) ) with both
 * fp32 operations rounded to nearest (for integer or half-integer z this is the correctly rounded
 * s*(q-z), the dequantisation of Eq. 1 / Eq. 5).  Bit-exact and deterministic. */
int slim_dequant(const void* packed, const uint8_t* bits_host, const void* scales, const void* zeros,
                 void* W, int N, int K, int g, void* stream);

/* Decode path, 1 <= M <= 16:  y = x * W-hat^T, fp32 accumulation, fp16 output (the paper's
 * inference kernel, App. B.2: group-by-group dequantisation and dot product with the shared
 * activation).  Streams the packed slices once; HBM-bound.  Results are deterministic for a
 * given (shape, device, workspace size).  x with Inf/NaN gives unspecified y.  `workspace` must be at least
 * 256 bytes (the kernel itself keeps its partial sums in shared memory).
 * A layer whose packed codes take 32 MB or more is run by the kernels of slim_mpq_gemv_set instead (same result
 * within the rounding of the accumulation order; at M = 1 with the fixed-point x described there) when the
 * workspace has the slim_workspace_bytes() that shape asks for; with a smaller workspace it takes the per-layer
 * kernel.  The call reads no host memory after it returns and can be captured in a CUDA graph either way.
 * At M = 1 every route takes x in the 22-bit fixed-point form described at slim_mpq_gemv_set (the per-layer
 * single-token kernel, CTAs that hold the whole K of a few 16-row tiles, serves the layers whose K fits a CTA's
 * shared memory with all CTAs resident at once; the others, and M > 1, multiply the fp16 x as it is).
 * The per-layer kernels are launched with programmatic stream serialisation and fetches packed, scales and zeros
 * before it waits for the kernel ahead of it on the stream: those three buffers must be complete when the call is
 * enqueued, or be written by a kernel that does not signal programmatic launch completion early (x and y may be
 * produced and consumed by the neighbouring kernels as usual).  At M = 1 the two kernels of the 32 MB route are launched
 * the same way, but touch no buffer before they have waited for the kernel ahead of them. */
int slim_mpq_gemv(const void* x, const void* packed, const uint8_t* bits_host,
                  const void* scales, const void* zeros, void* y,
                  int M, int N, int K, int g,
                  void* workspace, size_t workspace_bytes, void* stream);

/* Host-only introspection: the launch plan of slim_mpq_gemv's general kernel (M >= 2, and the single-token layers whose
 * K does not fit the single-token kernel) for this shape on the current device
 * (148 SMs assumed when no device is present).  out6 = {16-row tiles per CTA, k-slices =
 * cluster size, row blocks, dynamic shared memory bytes, 8-token MMA tiles, groups per chunk}.
 * grid = k-slices x row blocks, 8 warps per CTA. */
int slim_gemv_plan(int M, int N, int K, int g, const uint8_t* bits_host, int* out6);

/* Batched / prefill path, M > 16: same contract, tensor-core (tcgen05) kernel.  Zero points that
 * are multiples of 1/16 in [-16, 16) (every zero point Eq. 1 or Eq. 2 produces) are applied exactly,
 * others are rounded (to the nearest 1/16 at worst).  Deterministic for a given (shape, device, workspace size). */
int slim_mpq_gemm(const void* x, const void* packed, const uint8_t* bits_host,
                  const void* scales, const void* zeros, void* y,
                  int M, int N, int K, int g,
                  void* workspace, size_t workspace_bytes, void* stream);

/* slim_mpq_gemm for callers that must not allocate device memory.  (The paper has no counterpart
 * of this entry point; it exists for deployment.)  Typical callers: the enqueue callback of an
 * inference-engine plugin, which is handed input and output pointers and a stream and nothing
 * else, and serving loops whose memory budget was handed out at start-up, where a cudaMalloc would
 * stall every stream of the device or fail late.  Such callers have no workspace to pass.
 *
 * Same arithmetic and arguments as slim_mpq_gemm, except that the scratch (status word, stream-K
 * flags and fp32 partial tiles) is a fixed array inside the library: SLIM_STATIC_SCRATCH_MAX bytes
 * of device memory on every GPU that loads the library, held until the process exits.  The call
 * allocates and frees nothing.  A shape that would need more scratch on the current device (only
 * possible on a GPU with more than 148 SMs) returns SLIM_ERR_STATIC_SCRATCH and enqueues nothing.
 *
 * All calls on a device share that array.  Each call first clears the control words on `stream`,
 * then runs; two calls whose kernels can overlap on the GPU (different streams, no ordering) race
 * on it and give undefined results, so keep the calls of a device on one stream or order them.
 * The first call on each device looks up the array's device address (a driver query, no
 * allocation); make that first call outside any stream capture.  The array is reserved when the
 * library's device code is loaded on a GPU, which with lazy module loading is the first use of the
 * library there: make one call (of any entry point) at start-up, before memory gets tight.
 *
 * status_out: optional device pointer to one 32-bit word (4-byte aligned, may be NULL).  After
 * the work of a successful call completes (the no-op shapes included) it holds 0, or 1 if a
 * device-side wait gave up (y is then undefined);
 * it plays the part slim_workspace_status plays for a caller-owned workspace. */
#define SLIM_STATIC_SCRATCH_MAX (1280 + 148 * 256 * 128 * 4)
int slim_mpq_gemm_static(const void* x, const void* packed, const uint8_t* bits_host,
                         const void* scales, const void* zeros, void* y,
                         int M, int N, int K, int g, unsigned int* status_out, void* stream);

/* ---- layer-set launch of the decode path --------------------------------------------------- */

/* Several INDEPENDENT layers of the decode path (1 <= M <= SLIM_GEMV_SET_MAX_M = 64 tokens each) in one launch: the q/k/v or
 * gate/up projections that share an input, or a sweep over a model's layers.  (The paper launches
 * its kernel per layer, App. B.2; a decode-sized layer is too small to keep HBM busy on its own,
 * so the set is walked by persistent CTAs that stream the packed slices of one 128-row block after
 * another through a ring of shared-memory slots, with no pause between layers.)  No layer of a set
 * may read what another layer of the same set writes.
 *
 * Every layer gets the y = x * W-hat^T of slim_mpq_gemv (same products, fp32 accumulation in a
 * different order: the groups of a layer are added sorted by bit-width, and a set with fewer row blocks
 * than persistent CTAs adds them in up to 8 parts; fp16 output); the results are deterministic for a
 * given (set, device).
 * A set in which EVERY layer has M = 1 runs on integer tensor-core instructions: per group of 128
 * columns x is first rounded to fixed point with 22 bits relative to the group's largest |x_k|, so an
 * fp16 activation within a factor 2^11 of that maximum is taken exactly and a smaller one with an error
 * of at most 2^-22 of the maximum; the sums over the group are then exact.  Per output row n this adds at
 * most  sum over groups of 2^-22 max|x_group| sum_{k in group} |w-hat[n][k]|  to the error of the fp16
 * path at more than one token; x must be finite.  Sets with more tokens multiply
 * the fp16 x as it is, in MMA tiles of 8 tokens: the set's widest layer, rounded up to 8, 16, 32 or 64 tokens, fixes
 * how many tiles every layer computes, so a set is fastest when its layers have about the same token count.  (Between
 * 17 and about 100 tokens a layer set streams several times the weights per second that slim_mpq_gemm dequantises,
 * which is built for hundreds of tokens and more.)
 * N > 0 a multiple of 16, K > 0 a multiple of 128; g in {128, 256, 512}, one value for the whole set (for 256 and
 * 512 "group" in the bound above reads "128 columns of a group"); SLIM_ERR_UNSUPPORTED for 32 and 64. */
typedef struct slim_layer {
    const void* x;             /* device fp16 [M][K] */
    const void* packed;        /* device, packed codes of the layer */
    const void* scales;        /* device fp16 [G][N] */
    const void* zeros;         /* device fp16 [G][N] */
    void* y;                   /* device fp16 [M][N] */
    const uint8_t* bits_host;  /* host [K/g] */
    int M, N, K;
} slim_layer;

/* Filled by slim_gemv_set_plan, read by slim_mpq_gemv_set; plain data owned by the caller. */
typedef struct slim_gemv_set_info {
    int n_layers;
    int grid;              /* persistent CTAs */
    int n_slots;           /* ring slots per CTA */
    int slot_bytes;
    int token_tiles;       /* 8-token MMA tiles: 1, 2, 4 or 8 */
    int stage_tasks;       /* (layer, token, group) triples staged; layers with one x and one bit map count once */
    int n_items;           /* row blocks (work items) of the set */
    int max_bits;          /* widest group of the set */
    int max_tokens;        /* largest M of the set */
    int tiles_per_warp;    /* 16-row tiles a consumer warp owns (2): an item is 128 rows times this */
    int split;             /* parts the groups of a row block are cut into when the set has fewer row blocks than
                              persistent CTAs (1 .. 8; layers with few groups get fewer): fp32 partial outputs in the
                              workspace, added in part order by the warp whose part lands last */
    int n_counters;        /* arrival counters of the split row blocks (workspace, cleared by every launch) */
    int resident_pairs;    /* > 0: a small single-token set that runs as ONE launch with every CTA resident at once (the
                              whole K of 2 x resident_pairs row tiles per CTA, no ring, no staging kernel); the ring
                              fields above are then unused.  0: the persistent ring */
    int resident_cluster;  /* CTAs that share the staging of x in that launch (8 or 4) */
    size_t plan_bytes;
    size_t workspace_bytes;
    size_t resident_smem;  /* dynamic shared memory of that launch */
} slim_gemv_set_info;

/* Host-only.  Sizes of the device plan buffer and of the workspace a set needs on the current
 * device.  The workspace holds the status word and, per layer, its activations in tensor-core
 * fragment order. */
int slim_gemv_set_bytes(const slim_layer* layers_host, int n_layers, int g,
                        size_t* plan_bytes, size_t* workspace_bytes);

/* Validates the set, deals the work items to the persistent CTAs (heaviest item first, each to the
 * CTA with the least work so far, so the CTAs finish together) and writes the plan (layer
 * descriptors, every CTA's list of items) into `plan` (device, 16-byte aligned, plan_bytes from
 * slim_gemv_set_bytes) with copies enqueued on `stream`; fills *info.  layers_host and the bit
 * maps are read during the call only.  The plan stays valid while the layers' pointers do.
 * SLIM_ERR_UNSUPPORTED if the host-side lists of the deal cannot be allocated. */
int slim_gemv_set_plan(const slim_layer* layers_host, int n_layers, int g,
                       void* plan, size_t plan_bytes, slim_gemv_set_info* info, void* stream);

/* Runs the set: one small kernel puts every layer's activations into fragment order in the
 * workspace, one persistent kernel computes all layers (a small single-token set whose CTAs are all resident at
 * once runs as one launch instead: slim_gemv_set_info.resident_pairs; that launch uses programmatic stream
 * serialisation and requests packed, scales and zeros before it waits for the kernel ahead of it on the stream, under
 * the rule stated at slim_mpq_gemv).  `workspace` as for slim_mpq_gemv
 * (zeroed once with slim_workspace_init; slim_workspace_status reports a device-side time-out). */
int slim_mpq_gemv_set(const slim_gemv_set_info* info, const void* plan,
                      void* workspace, size_t workspace_bytes, void* stream);

/* ---- producing the inputs of the layer (the steps right before packing) ------------------- */

/* Group salience S_j = sum_{k in group j} a_k^2 * sum_n W[n][k]^2 (diagonal form of Definition 1 /
 * Theorem 1; first step of SBA in Algorithm 2).  W fp16 [N][K] device, act_norm fp32 [K] device,
 * salience fp64 [G] device.  fp64 accumulation in a fixed order. */
int slim_group_salience(const void* W, const float* act_norm, double* salience,
                        int N, int K, int g, void* stream);

/* Host-only.  Bit-width per group under |G_{N-1}| = |G_{N+1}| = p (Eq. 4): the p most salient
 * groups get avg_bits+1, the p least salient avg_bits-1, the rest avg_bits; equal salience ranks
 * the lower index higher.  p < 0 selects floor(G/4).  avg_bits in {2,3}. */
int slim_allocate_bits(const double* salience_host, int G, int avg_bits, int p, uint8_t* bits_host_out);

/* Asymmetric min-max quantizer of Eq. 1 per (row, group), in fp64 from the fp16 weights:
 * range extended to contain 0, s rounded to fp16 first (0 -> 1, overflow -> 65504),
 * z = clamp(-rint(lo/s)), q = clamp(rint(w/s) + z), rint = round-half-to-even.
 * W fp16 [N][K]; codes uint8 [N][K]; scales, zeros fp16 [G][N]; all device. */
int slim_quantize_minmax(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                         int N, int K, int g, void* stream);

/* slim_quantize_minmax restricted to the groups listed in groups_host[n_groups] (host, distinct
 * indices): only their columns of `codes` and their rows of `scales` and `zeros` are written,
 * under bits_host.  Used by the SBA search, whose consecutive candidates differ in two groups. */
int slim_quantize_minmax_groups(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                                int N, int K, int g, const int* groups_host, int n_groups, void* stream);

/* slim_quantize_minmax with the binarisation of Eq. 2 for the one-bit groups: q = [w >= 0]
 * (sign(0) = +1), alpha = mean |w| of the (row, group), stored as s = fp16(2 alpha), z = 1/2, so
 * that s (q - z) = +-alpha.  Groups of two or more bits use Eq. 1 as above.  Same layouts. */
int slim_quantize_minmax_sign1(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                               int N, int K, int g, void* stream);

/* Salience-Weighted Quantizer Calibration (Sec. 3.3, Eq. 5; function SQC of Algorithm 2), per
 * (row, group): for tau_i = 1 - lambda + i * lambda / n, i = 0 .. 2n-1, the quantizer
 * Delta = tau (w_max - w_min) / (2^b - 1), z = -round(tau w_min / Delta) is tried on the group and
 * the candidate with the smallest squared error (salient part, outside mu +- 3 sigma, plus the
 * rest; first candidate on ties) is kept, so the salient and the other weights share one scale
 * and one zero point.  Same storage conventions as slim_quantize_minmax (range extended to 0,
 * Delta rounded to fp16 first, z clamped to the code range); fp64 arithmetic with column-order
 * sums, so the result is reproducible bit for bit.  tau_index int32 [G][N] (device) receives the
 * chosen i and may be NULL.  The paper uses lambda = 0.1, n = 50; n <= 64. */
int slim_quantize_sqc(const void* W, const uint8_t* bits_host, uint8_t* codes, void* scales, void* zeros,
                      int* tau_index, int N, int K, int g, double lambda, int n, void* stream);

/* ---- Salience-Determined Bit Allocation (func SBA of Algorithm 2, Sec. 3.2.2, Eq. 4) --------- */

/* y = x * W^T in full precision: x fp16 [M][K], W fp16 [N][K], y fp32 [M][N] (device), fp32
 * accumulation (tensor cores).  The reference output "x w_f^T" of Eq. 4.  K a multiple of 32. */
int slim_dense_linear(const void* x, const void* W, float* y, int M, int N, int K, void* stream);

/* kl[t] = D_kl( softmax(y_ref[t]) || softmax(y_q[t]) ) for every token t (natural logarithm, softmax
 * over the N outputs of the token; the error measure of SBA, appendix on its evaluation function).
 * y_ref fp32 [M][N], y_q fp16 [M][N], kl fp64 [M], all device; fp64 arithmetic, fixed reduction order. */
int slim_softmax_kl(const float* y_ref, const void* y_q, double* kl, int M, int N, void* stream);

/* Host-only: bytes of workspace slim_sba_search needs (scratch of the layer calls, codes, scales, zeros,
 * packed buffer, both outputs, one error per candidate and token). */
int slim_sba_workspace_bytes(int M, int N, int K, int g, int avg_bits, size_t* out_bytes);

/* The search: groups ranked by salience (slim_group_salience; equal salience: lower index first);
 * for p = 0 (only if include_uniform), 1, ..., floor(G/2) the p most salient groups get avg_bits+1
 * bits and the p least salient avg_bits-1, the weight is quantised with slim_quantize_minmax under
 * that map, packed, and x * W-hat^T is computed by slim_mpq_gemv / slim_mpq_gemm; the candidate's
 * error is the mean over the M calibration tokens of slim_softmax_kl against slim_dense_linear(x, W).
 * The first p with the smallest error wins (Algorithm 2 compares with '<').
 * W fp16 [N][K], x fp16 [M][K], act_norm fp32 [K]: device.  workspace: device, 256-byte aligned.
 * Outputs on the HOST: *p_star, bits_host_out[G], errors_host[candidates] (may be NULL).
 * The call synchronises `stream` (it returns results to the host).  avg_bits in {2, 3}. */
int slim_sba_search(const void* W, const void* x, const float* act_norm, int M, int N, int K, int g, int avg_bits,
                    int include_uniform, void* workspace, size_t workspace_bytes,
                    int* p_star_host, uint8_t* bits_host_out, double* errors_host, void* stream);

/* ---- GPTQ error compensation around the quantizer (Algorithm 1) ----------------------------- */

/* Host-only: bytes of workspace for T calibration tokens and an N x K layer (two K x K fp64
 * matrices, the fp64 running weights, one group of errors and of quantizer input and output).
 * slim_gptq_factor alone needs the size for N = 0. */
int slim_gptq_workspace_bytes(int T, int N, int K, int g, size_t* out_bytes);

/* First two steps of Algorithm 1: H = (1/T) sum_t x_t x_t^T, then the upper-triangular U with
 * U^T U = (H + lambda_abs I)^-1 (the Cholesky factor the algorithm calls H_in), obtained as the
 * inverse of the factor R of H + lambda_abs I = R R^T.  lambda > 0 is relative to the mean
 * diagonal: lambda_abs = lambda * mean(diag H) (the GPTQ convention; the scale of H then does not
 * matter).  An input channel that is zero in every token gets H_kk = 1 and dead[k] = 1.
 * x fp16 [T][K] device; U_out fp64 [K][K] device (lower triangle zero); dead_out uint8 [K] device
 * or NULL; workspace 256-byte aligned.  fp64, fixed summation order. */
int slim_gptq_factor(const void* x, int T, int K, double lambda, double* U_out, uint8_t* dead_out,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Main loop of Algorithm 1 under the bit map bits_host[K/g]: for every group b in order, the
 * CURRENT weights of the group, rounded once to fp16, are quantised with slim_quantize_sqc
 * (use_sqc != 0; lambda 0.1, n 50) or slim_quantize_minmax; then
 *     E = (w_b - s (q - z)) / U[b, b]      (right division by the diagonal block = times R[b, b]),
 *     w[:, after b] -= E * U[b, after b].
 * The running weights are fp64 (dead input channels start at zero).  W fp16 [N][K], x fp16 [T][K];
 * codes uint8 [N][K], scales and zeros fp16 [G][N] as for slim_quantize_minmax; w_running fp64
 * [N][K] receives the running weights after the last update and may be NULL.  All device.
 * Deterministic.  The work is enqueued on `stream`; nothing is synchronised. */
int slim_gptq_quantize(const void* W, const void* x, const uint8_t* bits_host, double lambda, int use_sqc,
                       uint8_t* codes, void* scales, void* zeros, double* w_running,
                       int N, int K, int T, int g, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SLIM_H_ */
