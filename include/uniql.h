/*
 * uniql.h -- C ABI of the UniQL inference hot path for NVIDIA B200 (sm_100a).
 *
 * The library evaluates the linear layers of a model compressed the UniQL way
 * (arXiv 2512.03383): 4-bit group-quantised weights whose rows / columns were
 * sorted offline by importance, so that the pruning rate chosen on the device
 * only TRUNCATES each matrix to its leading sorted channels (Section 3.4,
 * "Quantization and On-device Adaptive Pruning").  Where the paper unpacks,
 * slices and re-packs the INT4 tensors whenever the rate changes, here the
 * kept channels are kernel arguments: nothing is copied or re-packed.
 * The Q / K projections also apply the rotary embedding to the retained head
 * dimensions, each surviving pair using the frequency of its ORIGINAL index
 * (Section 3.2, MHSA paragraph and Figure 3a, "fused RoPE kernel").
 *
 * Conventions
 *  - Pointers are DEVICE pointers unless a comment says "host".  The caller owns
 *    every buffer; the library never frees or keeps caller memory.
 *  - All work is enqueued on `stream` (a cudaStream_t passed as void*); no call
 *    synchronises the device.
 *  - Every function returns a uniql_status.  Argument errors are detected on the
 *    host before anything is launched; nothing aborts or throws.
 *  - There is no CPU fallback: without a usable CUDA device calls return
 *    UNIQL_ERR_CUDA.
 *  - Decode launches (M <= 16) and the launches of the tensor-core kernel (M > 16, bf16) carry the
 *    programmatic-stream-serialization attribute: back-to-back calls on one stream overlap their launch
 *    set-up and first weight stages with the tail of the preceding one (1.6 us per decode launch, 2 - 4 us
 *    per tensor-core launch), while everything that can depend on the preceding kernel (activations,
 *    outputs, workspace, bias, positions, indices) is touched only after it has completed.  Packed weights,
 *    scales and zero-points must not be written by a call's immediate predecessor on the stream
 *    unless that predecessor is a plain kernel (which completes before its successor starts).
 *    uniql_set_option("pdl", 0) (or UNIQL_PDL=0 in the environment at load time) turns the attribute off.
 *
 * Weight format (the interchange format; benchmark configuration 1)
 *  - W is stored in nn.Linear orientation, W[N][K]: N output channels (rows),
 *    K input channels, y = x W^T.  The paper writes W in R^{D_in x D_out}
 *    (Section 3.1); this is its transpose.
 *  - packed_w: uint8 [N][K/2]; byte b of row n holds input channel 2b in its low
 *    nibble and 2b+1 in its high nibble.  16-byte aligned, K % 128 == 0.
 *  - scales, zeros: fp16 [N][K/128], one pair per group of 128 consecutive STORED
 *    input channels:  w(n,k) = scale(n,k/128) * (code(n,k) - zero(n,k/128)).
 *    The paper's symmetric quantiser (Section 3.4 equation, N=4, group 128) is
 *    the case code = clamp(round(W/s),-8,7) + 8, zero = 8.  zero may be any
 *    finite fp16 value.
 *
 * Activations: x[M][ldx] and y[M][ldy], fp16 or bf16 (same type for both), COMPACT:
 * column t of x multiplies the t-th retained input channel, column j of y is the
 * j-th retained output channel.  Accumulation is fp32, one rounding to the output
 * type at the end (after the rotary embedding where it applies).
 * Any ldx >= the retained input count is valid; for batches above 16 rows a pitch of whole 128-byte lines
 * (ldx a multiple of 64) is the fast one: the tensor-core kernel fetches x in boxes of 64 columns, and a box row
 * that straddles two lines costs a second request (measured 6 % on the Qwen2.5-7B down projection at M = 2048 with
 * 12312 retained inputs packed at ldx = 12312 against ldx = 12352).  bf16 activations are copied to fp16 on such a
 * pitch by the library itself.
 */
#ifndef UNIQL_H_
#define UNIQL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  UNIQL_OK = 0,
  UNIQL_ERR_NULL = 1,        /* a required pointer is NULL */
  UNIQL_ERR_SHAPE = 2,       /* a size is out of range or inconsistent */
  UNIQL_ERR_ALIGN = 3,       /* a pointer or leading dimension is not aligned as required */
  UNIQL_ERR_DTYPE = 4,       /* unknown uniql_dtype */
  UNIQL_ERR_UNSUPPORTED = 5, /* valid request that no kernel of the forced path covers */
  UNIQL_ERR_WORKSPACE = 6,   /* workspace too small (see uniql_workspace_bytes) */
  UNIQL_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired */
  UNIQL_ERR_CUDA = 8         /* a CUDA runtime call failed (sticky errors included) */
} uniql_status;

typedef enum { UNIQL_F16 = 0, UNIQL_BF16 = 1 } uniql_dtype;

/* Kernel selection, for A/B tests.  AUTO: fp16 batches of M <= 16 take the persistent decode kernel
 * (UNIQL_PATH_DECODE); where the input map lies on 4- but not on 8-channel boundaries (head dims 108 and 84 on the
 * input side of o_proj, 1740 of 2048 leading channels) a small kernel in front re-lays the activations on
 * 8-channel boundaries in the workspace, and batches of M <= 4 for which that is not possible (no room in the
 * workspace, blocks that do not start on 8-channel boundaries) take the streaming kernel (UNIQL_PATH_GEMV:
 * every warp copies its own share of the codes through a private shared-memory ring) when its rules hold (one
 * input family, every start / keep / period a multiple of 4, K a multiple of 512, x 8-byte aligned with ldx a
 * multiple of 4, scale and zero-point arrays 8-byte aligned); everything
 * else (M > 16, bf16) the tensor-core (prefill) kernel when its alignment rules hold (activations 16-byte
 * aligned with a row pitch that is a multiple of 8, input map a leading block or one family of per-head
 * blocks on 64-channel boundaries with keep % 8 == 0), otherwise the generic kernel. */
typedef enum { UNIQL_PATH_AUTO = 0, UNIQL_PATH_GENERIC = 1, UNIQL_PATH_DECODE = 2,
               UNIQL_PATH_PREFILL = 3, UNIQL_PATH_GEMV = 4 } uniql_path;

/* Channel map (host struct, copied by value at call time).
 * On-device pruning keeps the leading sorted channels of D_int, of every head's
 * D_hd and of D_s, never of D_h (Section 3.4).  Because heads are concatenated,
 * "leading channels of every head" is a periodic set; a map is a short list of
 * such families.  Family f keeps channels start + h*period + i for h < count,
 * i < keep (STORED coordinates).  The compact order is family after family, block
 * after block.  Families must be given in increasing, non-overlapping order.
 *   MLP intermediate, keep k:           {0, k, k, 1}
 *   V rows / o_proj columns, per head:  {0, D_hd, d', H}
 *   Q or K rows (symmetric sort, Algorithm 2: idx_sym = [argsort, D_hd/2+argsort],
 *     so each half head keeps its leading d'/2 rows):  {0, D_hd/2, d'/2, 2H}     */
#define UNIQL_MAX_FAMILIES 8
typedef struct { int32_t start, period, keep, count; } uniql_family;
typedef struct { int32_t n_fam; uniql_family fam[UNIQL_MAX_FAMILIES]; } uniql_chanmap;

/* One weight matrix of a multi-matrix call (host struct; pointers inside are device). */
typedef struct {
  const uint8_t* packed_w;      /* [N][K/2] */
  const void* scales;           /* fp16 [N][K/128] */
  const void* zeros;            /* fp16 [N][K/128] */
  const void* bias;             /* activation dtype [N] in STORED coordinates, or NULL */
  int32_t N;                    /* stored rows */
  int32_t k_out;                /* used when out_map is NULL: keep the leading k_out rows */
  const uniql_chanmap* out_map; /* host, or NULL */
  void* y;                      /* [M][ldy] */
  int32_t ldy;                  /* elements; >= number of retained rows */
} uniql_job;
#define UNIQL_MAX_JOBS 4

int uniql_version(void);                 /* major*10000 + minor*100 + patch */
const char* uniql_status_string(int status);

/* Force a kernel path for subsequent calls of this process (tests / A-B timing). */
int uniql_set_path(int path);

/* Tuning and test options of the process (one table of atomics, read by every launch; each option takes its
 * initial value from the environment variable UNIQL_<NAME IN CAPITALS> when the library is loaded).
 * UNIQL_ERR_SHAPE for an unknown name.  Options a caller may want:
 *   "pdl"              1 / 0: programmatic stream serialization on decode and tensor-core launches (default 1)
 *   "prefill_streamk"  -1 automatic, 0 never, 1 / 2 always: split the contraction of the output tiles of the last,
 *                      partly filled round of the tensor-core kernel over several thread blocks.  The parts of a tile
 *                      go to slots of their own and are added in block order (1; bit-reproducible: the automatic
 *                      choice where every tile is split), or into one sum per tile in the order in which the blocks
 *                      finish (2; the automatic choice where whole tiles follow the split ones).  Launches with at most
 *                      one tile for every two SMs may instead run a cluster of two blocks per tile, half of the
 *                      contraction each, the second block's sums added in the first one's shared memory (3 forces it
 *                      wherever it fits; bit-reproducible).  0 makes the results of that kernel reproducible bit for
 *                      bit in every case (every tile is summed by one block).
 *   "prefill_dual"     -1 / 0: above 256 tokens a tile of the tensor-core kernel takes both accumulators (512
 *                      tokens per de-quantised weight stage); 0 keeps tiles of 256 tokens; 1 forces tiles of 512 tokens
 *                      wherever M > 256 (tests: 2 the same without half tiles for the left-over round, 3 with them
 *                      wherever they fit)
 *   "prefill_helpers"  1 / 0: the de-quantiser warps of the tensor-core kernel share the epilogue of a block's last tile
 *   "decode_split_batch" batches of 9..16 rows: 2 (default) one launch that streams the quantised activations
 *                      beside the weights, where the integer path applies, else two launches over half the batch;
 *                      1 always two launches; 0 always one launch with the activations staged whole
 * The others steer the work split of the kernels and exist for the tests: "decode_kp", "decode_rp",
 * "decode_stages", "decode_narrow", "decode_xstream", "decode_xcluster", "decode_i8", "prefill_grid",
 * "prefill_convert", "gemv_first", "gemv_depth", and "wait_shift" (the poll limit of the barrier between the two
 * phases of the one-launch MLP is divided by 2^wait_shift, so that a test can make that wait run out). */
int uniql_set_option(const char* name, int value);

/* ---- storage helpers (Section 3.4: 4-bit codes; bit-exact integer work) ----
 * codes: uint8 [N][K], one code (0..15) per byte.  packed: uint8 [N][K/2].  K even. */
int uniql_pack_u4(const uint8_t* codes, int64_t N, int64_t K, uint8_t* packed, void* stream);
int uniql_unpack_u4(const uint8_t* packed, int64_t N, int64_t K, uint8_t* codes, void* stream);
/* Full de-quantised matrix w[N][K] in `dt` (diagnostic; the hot path never materialises it).
 * Computed as fp32 scale*(code-zero), rounded once. */
int uniql_dequant(const uint8_t* packed, const void* scales, const void* zeros, int64_t N, int64_t K,
                  int dt, void* w, void* stream);

/* 4-bit embedding table (Section 3.4 applies 4-bit quantisation to the embedding and output layers too):
 * out[m][0..K) = scale * (code - zero) of table row ids[m], in `dt`, rounded once; the output layer
 * (lm_head) is uniql_qlinear on a [V][K] matrix.  packed [V][K/2], scales / zeros fp16 [V][K/128];
 * ids device int32 [M], M <= 65535; out [M][ldo], ldo >= K.  An id outside [0, V) gives a row of zeros and,
 * when bad_id (device int, may be NULL) is given, sets *bad_id = 1; nothing is read out of bounds. */
int uniql_embed_rows(const uint8_t* packed, const void* scales, const void* zeros, int64_t V, int64_t K,
                     const int32_t* ids, int64_t M, int dt, void* out, int64_t ldo, int* bad_id, void* stream);

/* ---- workspace ----
 * The decode kernel may split the input channels over several thread blocks; partial sums
 * and arrival counters live in a workspace.  Calls without a workspace argument use a
 * per-device buffer the library allocates at its first use on that device (so the first
 * call on a device must not happen during stream capture).  A caller-provided workspace
 * must be 256-byte aligned, at least uniql_workspace_bytes() large, and prepared once by
 * uniql_workspace_init (zeroes the counters; they return to zero after every call).
 * Calls that share a workspace must not overlap on the device. */
/* For M > 16 (tensor-core path) the workspace carries the status word, for bf16 activations
 * an fp16 copy of x (M x K x 2 bytes): the tensor cores run on fp16 operands, because weights rounded
 * to bf16 would alone spend the 2e-3 error budget; bf16 magnitudes beyond 65504 saturate.  When the
 * workspace is too small for the copy the tiles are converted inside the kernel (same result, slower).
 * It also carries the fp32 parts of output tiles whose contraction is split over several thread blocks
 * (fewer than two slots of 128 rows x 256 or 512 tokens per SM).  Where every tile is split the parts are added in block order; where
 * split tiles stand in front of whole tiles they are added in the order in which the blocks finish, and with more
 * than two blocks on a tile the last bit of an fp32 sum, and rarely of the rounded output, can differ
 * between two runs on the same input; uniql_set_option("prefill_streamk", 0) switches the splitting off.  Activations below fp16's range are affected too: bf16 values under 2^-24 become zero
 * and those under 2^-14 lose significand bits in the fp16 copy.  Without room for the
 * sums every tile is computed by one block (reproducible, slower for shapes that fill few SMs). */
size_t uniql_workspace_bytes(int M, int K, int N_total);
int uniql_workspace_init(void* workspace, size_t bytes, void* stream);
/* Every wait inside the kernels is bounded.  When one expires the kernel stops early and writes
 * UNIQL_ERR_TIMEOUT into a status word of the workspace it ran with; the outputs of that call are
 * then incomplete.  This call synchronises the device and copies the word to *status (host):
 * UNIQL_OK when no wait has expired since the workspace was initialised.  workspace NULL = the
 * library's buffer of the current device. */
int uniql_workspace_status(void* workspace, int* status);

/* ---- the quantised, pruned linear layer (Section 3.4; decode and prefill of Section 5) ----
 * Simple form: fp16 x[M][k_in], fp16 y[M][k_out], keep the leading k_in input and k_out
 * output channels of the sorted matrix W[N][K].  k_in, k_out > 0, multiples of 4,
 * k_in <= K, k_out <= N, M >= 1. */
int uniql_qlinear(const void* x, const uint8_t* packed_w, const void* scales, const void* zeros,
                  int M, int K, int N, int k_in, int k_out, void* y, void* stream);

/* The same layer for callers that cannot allocate device memory (no counterpart in the paper: this
 * is a property of the library, not of the method).  Think of a serving process whose device memory
 * was handed out completely at start-up, a real-time loop in which cudaMalloc could stall on the
 * driver, or a sandbox in which the call is forbidden.  Nothing is allocated here, by this library or
 * by anything it calls: the scratch memory of the decode kernel is a fixed array of
 * UNIQL_NOALLOC_SCRATCH_BYTES inside the library's device image (every GPU that loads the library
 * carries it until the process ends).
 *  - Arguments as uniql_qlinear (fp16, leading k_in x k_out block); decode only: M <= 16, else
 *    UNIQL_ERR_UNSUPPORTED.  A problem whose split-K partial sums do not fit the fixed array returns
 *    UNIQL_ERR_WORKSPACE and launches nothing.  The need is 256 KB plus roughly 512 bytes per 64
 *    retained rows and batch row (more when large M * K splits the input channels over several
 *    groups of thread blocks); the Llama-3-8B MLP matrices fit for every M <= 16.  Batches of 9..16 rows take
 *    one launch here whatever option "decode_split_batch" says (streamed activations where they apply, else
 *    staged ones), and the small kernel that quantises streamed activations writes into the same array.
 *  - The first call on a device looks up the array's device address (once per device, with that
 *    device current); make that first call outside any stream capture.
 *  - All calls share the one array, and it keeps what the previous call left: each call clears the
 *    part that must start at zero on `stream` before it launches.  Two calls that may overlap on the
 *    GPU (different streams without ordering between them) race on it: order them. */
#define UNIQL_NOALLOC_SCRATCH_BYTES (8u << 20)
int uniql_qlinear_noalloc(const void* x, const uint8_t* packed_w, const void* scales, const void* zeros,
                          int M, int K, int N, int k_in, int k_out, void* y, void* stream);
/* Status of the uniql_qlinear_noalloc calls made so far on the current device (no counterpart in the paper
 * either: it belongs to the entry point above).  Every wait inside the kernel is bounded; a call whose wait
 * expired leaves UNIQL_ERR_TIMEOUT in a status word inside the fixed array and an incomplete y, while the call
 * itself, which only enqueues work, has long returned UNIQL_OK.  uniql_workspace_status cannot see that word.
 * This call waits for the device, copies the word to *status (host) and allocates nothing.  The next
 * uniql_qlinear_noalloc call clears the word before it launches: read it after the calls whose outcome matters
 * and before issuing more of them. */
int uniql_noalloc_status(int* status);

/* General form: dtype, leading dimensions, bias, channel maps (NULL map = leading k).
 * x and y must be 4-byte aligned with even ldx / ldy; every family's start and keep must be
 * multiples of 4.  workspace may be NULL (library buffer). */
int uniql_qlinear_ex(const void* x, int ldx, int dt, const uint8_t* packed_w, const void* scales,
                     const void* zeros, const void* bias, int M, int K, int N,
                     const uniql_chanmap* in_map, int k_in, const uniql_chanmap* out_map, int k_out,
                     void* y, int ldy, void* workspace, size_t ws_bytes, void* stream);

/* Several matrices that share x, M, K and the input map in ONE launch (gate|up, q|k|v).
 * jobs: host array of n_jobs <= UNIQL_MAX_JOBS entries. */
int uniql_qlinear_multi(const void* x, int ldx, int dt, int M, int K, const uniql_chanmap* in_map,
                        int k_in, int n_jobs, const uniql_job* jobs, void* workspace, size_t ws_bytes,
                        void* stream);

/* ---- fused Q and K projection + rotary embedding on the retained head dims ----
 * (Section 3.2 MHSA paragraph, Figure 3a; GQA index sharing: Algorithm 6.)
 * Wq[n_q_heads*head_dim][K] and Wk[n_kv_heads*head_dim][K] are symmetric-sorted per head;
 * each head keeps head_keep dims: rows [0, head_keep/2) of both of its halves.
 * q_out[M][n_q_heads*head_keep], k_out[M][n_kv_heads*head_keep]; inside a head the order is
 * [first-half survivors | second-half survivors].  Compact pair c = (column c, column
 * c + head_keep/2) of query head h is rotated by angle pos[m] * inv_freq[p] with
 * p = retained_idx[h / (n_q_heads/n_kv_heads)][c], the ORIGINAL pair index (only half of the
 * symmetric index vector is stored), inv_freq[p] = theta^(-2p/head_dim) unless a table is
 * given:  (a, b) -> (a cos - b sin, b cos + a sin), applied to the fp32 accumulators (bias
 * included) before the single output rounding.
 *   retained_idx: device int32 [n_kv_heads][head_keep/2], values in [0, head_dim/2)
 *   pos:          device int32 [M]
 *   inv_freq:     HOST double [head_dim/2] or NULL
 * head_dim even, <= 256; head_keep even, 2 <= head_keep <= head_dim; n_q_heads % n_kv_heads == 0.
 * Index values are not range-checked on the host (they live on the device); the kernels
 * clamp them into [0, head_dim/2). */
int uniql_qk_rope_proj(const void* x, int ldx, int dt, const uint8_t* wq, const void* sq,
                       const void* zq, const uint8_t* wk, const void* sk, const void* zk,
                       const void* bq, const void* bk, int M, int K, int n_q_heads, int n_kv_heads,
                       int head_dim, int head_keep, const int32_t* retained_idx, const int32_t* pos,
                       double theta, const double* inv_freq, void* q_out, int ldq, void* k_out,
                       int ldk, void* workspace, size_t ws_bytes, void* stream);

/* ---- Q, K and V projections of one attention block in ONE launch ----
 * (Section 3.2, MHSA paragraph: the weights of a head form the groups {W_q, W_k}, sorted symmetrically and
 * rotated, and {W_v, W_o}, sorted per head without the symmetry constraint.)  As uniql_qk_rope_proj, plus
 * Wv[n_kv_heads*head_dim][K] as a third matrix of the same launch: every key-value head keeps its leading
 * v_keep rows, no rotation, v_out[M][n_kv_heads*v_keep] (row h*v_keep + r = stored row h*head_dim + r).
 * v_keep a multiple of 4, 4 <= v_keep <= head_dim; bv optional.  All three share x, so x is staged once and
 * the three weight matrices stream through one launch. */
int uniql_qkv_rope_proj(const void* x, int ldx, int dt, const uint8_t* wq, const void* sq, const void* zq,
                        const uint8_t* wk, const void* sk, const void* zk, const uint8_t* wv,
                        const void* sv, const void* zv, const void* bq, const void* bk, const void* bv,
                        int M, int K, int n_q_heads, int n_kv_heads, int head_dim, int head_keep,
                        int v_keep, const int32_t* retained_idx, const int32_t* pos, double theta,
                        const double* inv_freq, void* q_out, int ldq, void* k_out, int ldk, void* v_out,
                        int ldv, void* workspace, size_t ws_bytes, void* stream);

/* ---- SwiGLU MLP block:  y = ( silu(x Wg^T) * (x Wu^T) ) Wd^T ----
 * (Section 3.2, MLP paragraph: f_MLP(X) = (sigma(X W_g) . X W_u) W_d with sigma(t) = t / (1 + exp(-t)),
 * the gate of the Llama / Qwen blocks the paper compresses; Section 3.4: after sorting, pruning the
 * intermediate dimension keeps the leading k_int channels.)
 * Stored matrices: Wg, Wu [inter][hidden] and Wd [hidden][inter] packed as for uniql_qlinear, scales /
 * zeros [rows][cols/128] fp16.  Used: rows [0, k_int) of Wg and Wu, columns [0, k_int) of Wd.
 *   x [M][ldx] fp16 (hidden columns),  h [M][ldh] fp16 (k_int columns: the gated activations, rounded to
 *   fp16 once; written by the call, valid on return),  y [M][ldy] fp16 (hidden columns).
 * fuse = 1: ONE launch (gate|up tiles, a grid-wide barrier with a bounded wait, down tiles; weights of the
 *   down projection are prefetched across the barrier); UNIQL_ERR_UNSUPPORTED when M > 8 or the staged
 *   activations do not fit in shared memory.  fuse = 0: two launches (gate|up with the gated product as
 *   epilogue, then down).  fuse = -1: the faster of the two on this hardware (two launches: the boundary
 *   between dependent launches costs less than the grid-wide barrier).  M in 9..16: each of the two launches
 *   streams its quantised activations beside the weights (option "decode_split_batch" 1: two halves of the batch).
 * Limits at 1 <= M <= 16: fp16; hidden, inter multiples of 256; k_int a multiple of 8; ldx, ldh multiples
 * of 8; x and h 16-byte aligned.  Other shapes: UNIQL_ERR_UNSUPPORTED (compose uniql_qlinear_multi calls).
 * M > 16 (the name is historical): two launches of the tensor-core kernel.  The first takes Wg and Wu as a
 *   pair, retained row i of each in neighbouring rows of every tile, and stores silu(g) * u as h; the second
 *   is the down projection over the leading k_int channels of h (on the generic kernel when ldh is not a
 *   multiple of 8 or h is not 16-byte aligned).  fp16; hidden, inter multiples of 128; any k_int in
 *   [1, inter]; ldx a multiple of 8 and x 16-byte aligned; fuse = 1 is UNIQL_ERR_UNSUPPORTED.
 * workspace: NULL (library buffer) or uniql_mlp_workspace_bytes(M, hidden, inter) bytes, zeroed once by
 * uniql_workspace_init; after a UNIQL_ERR_TIMEOUT status it must be zeroed again before reuse. */
size_t uniql_mlp_workspace_bytes(int M, int hidden, int inter);
/* The same block for either activation type and any M: dt = UNIQL_F16 with M <= 16 is
 * uniql_mlp_swiglu_decode(fuse = -1); everything else (M > 16, and bf16 at any M) takes the two launches of
 * the tensor-core kernel described above, x, h and y all of type dt (bf16: the tensor cores run on an fp16
 * copy of x and of h, as for uniql_qlinear; h is rounded to bf16 once).  Same argument meaning and errors. */
int uniql_mlp_swiglu(const void* x, int ldx, int dt, const uint8_t* wg, const void* sg, const void* zg,
                     const uint8_t* wu, const void* su, const void* zu, const uint8_t* wd, const void* sd,
                     const void* zd, int M, int hidden, int inter, int k_int, void* h, int ldh, void* y,
                     int ldy, void* workspace, size_t ws_bytes, void* stream);
int uniql_mlp_swiglu_decode(const void* x, int ldx, const uint8_t* wg, const void* sg, const void* zg,
                            const uint8_t* wu, const void* su, const void* zu, const uint8_t* wd,
                            const void* sd, const void* zd, int M, int hidden, int inter, int k_int,
                            void* h, int ldh, void* y, int ldy, int fuse, void* workspace,
                            size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* UNIQL_H_ */
