// Internal structures and device helpers shared by the UniQL kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/uniql.h"

namespace uniql {

constexpr int kGroup = 128;       // quantisation group along the input channels (Section 3.4)
constexpr int kMaxFam = UNIQL_MAX_FAMILIES;
constexpr int kMaxJobs = UNIQL_MAX_JOBS;
constexpr int kMaxHalfDim = 128;  // head_dim/2 <= 128

struct Fam { int start, period, keep, count; };

// A channel map with the compact offset of every family precomputed.
struct ChanMap {
  int n_fam;
  int total;            // number of retained channels
  Fam fam[kMaxFam];
  int base[kMaxFam];    // compact index of the family's first channel
};

// Rotary-embedding description of a job (Section 3.2, fused RoPE with index gather).
struct RopeDesc {
  int enabled;
  int n_heads;      // heads of THIS matrix (query heads for Wq, kv heads for Wk)
  int rep;          // query heads per kv head (1 for Wk)
  int head_dim;     // un-pruned D_hd
  int head_keep;    // retained dims per head (even)
};

struct JobDev {
  const uint8_t* w;
  const __half* scales;
  const __half* zeros;
  const void* bias;
  void* y;
  int ldy;
  int N;
  int k_out;          // retained rows
  ChanMap omap;       // ignored when rope.enabled (rows follow the half-head rule)
  RopeDesc rope;
  int pair;           // tensor-core kernel only.  1: the gate matrix of a SwiGLU pair (Section 3.2, MLP paragraph):
                      // rows 2i, 2i+1 of a tile are retained row i of this matrix and of the NEXT job's (the up
                      // matrix), and the epilogue stores silu(g_i) * u_i at column i of this job's output.
                      // 2: that next job (it has no tiles of its own).
};

struct Params {
  const void* x;
  int ldx;
  int dt;             // uniql_dtype
  int M;
  int K;              // stored input channels
  int k_in;           // retained input channels
  ChanMap imap;
  int n_jobs;
  JobDev job[kMaxJobs];
  const int32_t* idx;   // [n_kv_heads][head_keep/2] original pair indices
  const int32_t* pos;   // [M]
  unsigned long long rope_turn[kMaxHalfDim];   // frac(inv_freq / 2 pi) * 2^64, per original pair
};

// ---------------------------------------------------------------- channel-map arithmetic
// compact index -> stored index
__host__ __device__ inline int map_compact_to_stored(const ChanMap& m, int j) {
  int f = 0;
  while (f + 1 < m.n_fam && j >= m.base[f + 1]) ++f;
  int r = j - m.base[f];
  int h = r / m.fam[f].keep;
  return m.fam[f].start + h * m.fam[f].period + (r - h * m.fam[f].keep);
}

// stored index -> compact index, or -1 when the channel is pruned
__host__ __device__ inline int map_stored_to_compact(const ChanMap& m, int k) {
  for (int f = 0; f < m.n_fam; ++f) {
    const Fam& a = m.fam[f];
    if (k < a.start) return -1;
    int r = k - a.start;
    int h = r / a.period;
    if (h >= a.count) continue;
    int o = r - h * a.period;
    return (o < a.keep) ? m.base[f] + h * a.keep + o : -1;
  }
  return -1;
}

// Output row `j` (compact order) of a rope job: head h, half s, position c inside the half.
// Compact layout per head: [first-half survivors | second-half survivors] (Section 3.2).
struct RopeRow { int stored; int head; int c; int is_hi; };
__host__ __device__ inline RopeRow rope_row(const RopeDesc& r, int j) {
  RopeRow o;
  int half = r.head_keep >> 1;
  o.head = j / r.head_keep;
  int within = j - o.head * r.head_keep;
  o.is_hi = within >= half;
  o.c = within - (o.is_hi ? half : 0);
  o.stored = o.head * r.head_dim + (o.is_hi ? (r.head_dim >> 1) : 0) + o.c;
  return o;
}

// ---------------------------------------------------------------- dtype helpers
template <typename T> struct DT;
template <> struct DT<__half> {
  using T2 = __half2;
  static __device__ inline float to_f(__half v) { return __half2float(v); }
  static __device__ inline __half from_f(float v) { return __float2half_rn(v); }
  static __device__ inline float2 to_f2(__half2 v) { return __half22float2(v); }
};
template <> struct DT<__nv_bfloat16> {
  using T2 = __nv_bfloat162;
  static __device__ inline float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ inline __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
  static __device__ inline float2 to_f2(__nv_bfloat162 v) { return __bfloat1622float2(v); }
};

// ---------------------------------------------------------------- rotary angle
// cos / sin of pos * inv_freq.  The product reaches thousands of radians, where an fp32
// product alone would already be off by ~1e-3 rad.  The host therefore passes each frequency
// as a 64-bit fixed-point fraction of a turn (turn = frac(inv_freq / 2 pi) * 2^64): the
// integer product pos * turn wraps modulo one turn by itself, exactly, and its upper 32 bits,
// read as a signed number, are the reduced angle in [-1/2, 1/2) turns with 2^-32 resolution.
// The fast fp32 intrinsics then work on an argument in [-pi, pi).  (fp64 arithmetic here cost
// the 64 x 256 angles of one tensor-core tile about as much time as the tile's main loop.)
__host__ inline unsigned long long rope_turn_of(double inv_freq) {
  long double t = (long double)inv_freq / 6.283185307179586476925286766559L;
  t -= floorl(t);
  const long double scaled = t * 18446744073709551616.0L;
  return scaled >= 18446744073709551615.0L ? ~0ull : (unsigned long long)scaled;
}
__device__ inline void rope_cos_sin(int pos, unsigned long long turn, float& c, float& s) {
  const unsigned long long a = (unsigned long long)(long long)pos * turn;
  const float af = (float)(int)(a >> 32) * (6.283185307179586476925286766559f / 4294967296.f);
  c = __cosf(af);
  s = __sinf(af);
}

// Tuning / test options of the process (uniql_set_option); every launch reads them from one table of atomics.
enum OptId {
  kOptPdl = 0, kOptDecodeKp, kOptDecodeRp, kOptDecodeStages, kOptDecodeNarrow, kOptDecodeXstream, kOptDecodeXcluster,
  kOptDecodeI8, kOptDecodeSplitBatch, kOptPrefillGrid, kOptPrefillConvert, kOptPrefillStreamk, kOptPrefillDual, kOptPrefillHelpers, kOptGemvFirst,
  kOptGemvDepth, kOptWaitShift, kOptCount
};
int opt(int id);

// host launchers (one per kernel file) --------------------------------------------------
struct LaunchCfg {
  void* workspace;
  size_t ws_bytes;
  cudaStream_t stream;
  int clear_header;      // decode kernel: zero the arrival counters of the launch and the status block on `stream`
                         // once the launch is certain (a workspace that may hold what an unfinished call left)
};
int launch_generic(const Params& p, const LaunchCfg& cfg);
// out[m][h * keep8 + r] = r < keep ? x[m][h * keep + r] : 0  (2-byte elements; out 16-byte aligned, keep8 % 8 == 0)
int launch_relay_x(const void* x, long long ldx, int M, int count, int keep, int keep8, void* out, cudaStream_t stream);
int launch_decode(const Params& p, const LaunchCfg& cfg);
int decode_supported(const Params& p);
int decode_integer_path(const Params& p);
int decode_streams_batch(const Params& p);   // its int8 path takes the input map (8-channel boundaries)
size_t decode_workspace_bytes(int M, int K, int N_total);
int decode_status_offset();   // byte offset of the device status word inside a workspace
size_t decode_workspace_header_bytes();   // counters + status word: the part that must start at zero
// SwiGLU MLP at decode (Section 3.2, MLP paragraph: y = (silu(x Wg^T) * (x Wu^T)) Wd^T with the trailing `inter - k_int`
// sorted intermediate channels pruned): leading k_int rows of Wg, Wu and leading k_int columns of Wd.
struct MlpDecode {
  const void* x; int ldx;      // [M][hidden] fp16
  int M, hidden, inter, k_int;
  const uint8_t *wg, *wu, *wd; // packed [inter][hidden/2], [inter][hidden/2], [hidden][inter/2]
  const __half *sg, *zg, *su, *zu, *sd, *zd;
  void* h; int ldh;            // [M][k_int] fp16: the gated activations (written, then read)
  void* y; int ldy;            // [M][hidden] fp16
};
// fuse != 0: both products in one launch (UNIQL_ERR_UNSUPPORTED when the shapes do not allow it);
// fuse == 0: two launches.
int launch_mlp_decode(const MlpDecode& d, int fuse, const LaunchCfg& cfg);
int mlp_decode_supported(const MlpDecode& d);
size_t mlp_decode_workspace_bytes(int M, int hidden, int inter);
// streaming kernel for one to four rows (csrc/gemv.cu)
int launch_gemv(const Params& p, const LaunchCfg& cfg);
int gemv_supported(const Params& p);
size_t gemv_workspace_bytes(int M, int K, int N_total);
int launch_gemv_mlp(const MlpDecode& d, const LaunchCfg& cfg);
int gemv_mlp_supported(const MlpDecode& d);
int launch_prefill(const Params& p, const LaunchCfg& cfg);
int prefill_supported(const Params& p);
size_t prefill_workspace_bytes(int M, int K);

}  // namespace uniql
