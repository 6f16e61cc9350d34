// Host side of the C ABI: argument validation, channel-map compilation, workspace handling
// and the dispatch by M between the decode, prefill and generic kernels.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

using namespace uniql;

namespace {

std::atomic<int> g_path{UNIQL_PATH_AUTO};

// name, environment variable read once at load, default
struct OptDesc { const char* name; const char* env; int dflt; };
const OptDesc kOpts[kOptCount] = {
    {"pdl", "UNIQL_PDL", 1},                            // programmatic stream serialization (decode and tensor-core launches)
    {"decode_kp", "UNIQL_DECODE_KP", 0},                // groups of blocks over the input channels (0: automatic)
    {"decode_rp", "UNIQL_DECODE_RP", 0},                // blocks per group (0: one per SM)
    {"decode_stages", "UNIQL_DECODE_STAGES", 0},        // ring stages (0: automatic)
    {"decode_narrow", "UNIQL_DECODE_NARROW", -1},       // narrow tiles: -1 automatic, 0 off, 1 on
    {"decode_xstream", "UNIQL_DECODE_XSTREAM", -1},     // streamed activations: -1 automatic, 0 off, 1 on
    {"decode_xcluster", "UNIQL_DECODE_XCLUSTER", -1},   // shared staging in clusters of two: -1 automatic, 0 off, 1 on
    {"decode_i8", "UNIQL_DECODE_I8", 1},                // integer path (0: fp16 MMAs)
    {"decode_split_batch", "UNIQL_DECODE_SPLIT_BATCH", 2},   // batches of 9..16: one streamed launch where it applies
    {"prefill_grid", "UNIQL_PREFILL_GRID", 0},          // blocks of the tensor-core kernel (0: one per SM)
    {"prefill_convert", "UNIQL_PREFILL_CONVERT_IN_KERNEL", 0},   // 1: bf16 tiles converted inside the kernel
    {"prefill_streamk", "UNIQL_PREFILL_STREAMK", -1},   // split tiles: -1 automatic, 0 never, 1 always (a slot per part), 2 always (one sum per tile), 3 pairs of blocks
    {"prefill_dual", "UNIQL_PREFILL_DUAL", -1},         // tiles of 512 tokens on both accumulators: -1 by cost, 0 never, 1 always (2 / 3: without / with half tiles)
    {"prefill_helpers", "UNIQL_PREFILL_HELPERS", 1},    // de-quantiser warps share the epilogue of a block's last tile
    {"gemv_first", "UNIQL_GEMV_FIRST", 0},              // 1: the streaming kernel wherever it applies (M <= 4)
    {"gemv_depth", "UNIQL_GEMV_DEPTH", 0},              // ring slots per warp of the streaming kernel (0: automatic)
    {"wait_shift", "UNIQL_WAIT_SHIFT", 0},              // bounded device waits: limits divided by 2^shift (tests)
};
std::atomic<int> g_opt[kOptCount];
const bool g_opt_init = [] {
  for (int i = 0; i < kOptCount; ++i) {
    const char* e = getenv(kOpts[i].env);
    g_opt[i].store(e ? atoi(e) : kOpts[i].dflt);
  }
  return true;
}();

constexpr int kMaxDevices = 64;
constexpr size_t kLibWorkspaceBytes = (size_t)192 << 20;
void* g_ws[kMaxDevices] = {nullptr};
std::mutex g_ws_mutex;

// Per-device library workspace, allocated (and its counters zeroed) at first use.
int lib_workspace(void** ws, size_t* bytes, cudaStream_t stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return UNIQL_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  if (!g_ws[dev]) {
    void* p = nullptr;
    if (cudaMalloc(&p, kLibWorkspaceBytes) != cudaSuccess) { cudaGetLastError(); return UNIQL_ERR_CUDA; }
    if (cudaMemset(p, 0, kLibWorkspaceBytes) != cudaSuccess) { cudaFree(p); return UNIQL_ERR_CUDA; }
    g_ws[dev] = p;
  }
  (void)stream;
  *ws = g_ws[dev];
  *bytes = kLibWorkspaceBytes;
  return UNIQL_OK;
}

// Validate a caller map against a dimension of size D and compile it.
int compile_map(const uniql_chanmap* src, int k_lead, int D, ChanMap* out) {
  memset(out, 0, sizeof(*out));
  if (!src) {
    if (k_lead <= 0 || k_lead > D) return UNIQL_ERR_SHAPE;
    out->n_fam = 1;
    out->fam[0] = Fam{0, k_lead, k_lead, 1};
    out->base[0] = 0;
    out->total = k_lead;
    return UNIQL_OK;
  }
  if (src->n_fam < 1 || src->n_fam > kMaxFam) return UNIQL_ERR_SHAPE;
  int64_t prev_end = 0, total = 0;
  for (int f = 0; f < src->n_fam; ++f) {
    const uniql_family& a = src->fam[f];
    if (a.start < 0 || a.keep <= 0 || a.count <= 0 || a.period <= 0) return UNIQL_ERR_SHAPE;
    if (a.count > 1 && a.period < a.keep) return UNIQL_ERR_SHAPE;
    int64_t end = (int64_t)a.start + (int64_t)(a.count - 1) * a.period + a.keep;
    if (a.start < prev_end || end > D) return UNIQL_ERR_SHAPE;
    prev_end = end;
    out->fam[f] = Fam{a.start, a.period, a.keep, a.count};
    out->base[f] = (int)total;
    total += (int64_t)a.keep * a.count;
  }
  if (total > D) return UNIQL_ERR_SHAPE;
  out->n_fam = src->n_fam;
  out->total = (int)total;
  return UNIQL_OK;
}

int check_common(const void* x, int ldx, int dt, int M, int K) {
  if (!x) return UNIQL_ERR_NULL;
  if (dt != UNIQL_F16 && dt != UNIQL_BF16) return UNIQL_ERR_DTYPE;
  if (M < 1 || K < kGroup || (K % kGroup) != 0 || ldx < 1) return UNIQL_ERR_SHAPE;
  if (((uintptr_t)x) & 1) return UNIQL_ERR_ALIGN;
  return UNIQL_OK;
}

int check_weight(const uint8_t* w, const void* s, const void* z, int N) {
  if (!w || !s || !z) return UNIQL_ERR_NULL;
  if (N < 1) return UNIQL_ERR_SHAPE;
  if ((((uintptr_t)w) & 15) || (((uintptr_t)s) & 1) || (((uintptr_t)z) & 1)) return UNIQL_ERR_ALIGN;
  return UNIQL_OK;
}

// The activations re-laid so that the fast kernels can read them: one input family whose kept blocks (or whose row
// pitch / base address) are not on 16-byte boundaries becomes the same family with every block padded to a multiple
// of 8 channels, the padding zero (the extra channels then meet real weights with zero activations).  Fills `q` with
// the parameters of the re-laid problem (x still to be set) and returns the padded block size, or 0 when the map
// does not allow it.
int relay_candidate(const Params& p, Params* q) {
  if (p.imap.n_fam != 1) return 0;
  const Fam& a = p.imap.fam[0];
  const int keep8 = (a.keep + 7) / 8 * 8;
  if ((a.start % 8) != 0) return 0;
  if (a.count > 1 && ((a.period % 8) != 0 || keep8 > a.period)) return 0;
  if (a.count == 1 && a.start + keep8 > p.K) return 0;
  *q = p;
  q->imap.fam[0].keep = keep8;
  q->imap.total = keep8 * a.count;
  q->imap.base[0] = 0;
  q->k_in = q->imap.total;
  q->ldx = q->imap.total;
  q->x = reinterpret_cast<const void*>((uintptr_t)256);     // (aligned as the workspace region will be)
  return keep8;
}

int dispatch(const Params& p_in, void* workspace, size_t ws_bytes, void* stream) {
  if (cudaPeekAtLastError() != cudaSuccess) return UNIQL_ERR_CUDA;
  LaunchCfg cfg{workspace, ws_bytes, (cudaStream_t)stream};
  int path = g_path.load();
  Params p = p_in;
  bool dec_ok = p.M <= 16 && decode_supported(p);
  // every batch the decode kernel does not take (more than 16 rows, bf16) goes to the tensor cores when the maps
  // allow it: at 17..63 rows the generic kernel measured 13 to 26 times slower (930 us against 71 us for the
  // Llama-3-8B gate|up at M = 17)
  bool pre_ok = prefill_supported(p);
  // One to four rows whose input map is on 4- but not 8-channel boundaries (head dims 108 and 84, 1740 of 2048
  // channels): re-laid on 8-channel boundaries for the decode kernel's integer path where that is possible (with
  // the small kernel in front under programmatic dependent launch: Llama-3-8B o_proj at head dim 108, M = 1 / 4:
  // 5.9 / 8.4 us), else the streaming kernel, which stages activations in 8-byte units (8.7 / 13.1 us).
  bool gv = path == UNIQL_PATH_GEMV || (path == UNIQL_PATH_AUTO && gemv_supported(p) && opt(kOptGemvFirst) == 1);
  const bool gv_else = path == UNIQL_PATH_AUTO && !gv && gemv_supported(p) && !(dec_ok && decode_integer_path(p));
  bool relaid = false;
  // Everything else that misses a fast kernel only because of where its activations lie (blocks of 108 or 84
  // channels, an odd row pitch) gets them re-laid in the workspace by a small kernel in front: 5..16 rows then run
  // on the integer path of the decode kernel, larger batches and bf16 on the tensor cores.
  if (!gv && path != UNIQL_PATH_GENERIC) {
    const bool decode_size = p.M <= 16 && p.dt == UNIQL_F16 && path != UNIQL_PATH_PREFILL;
    const bool slow = decode_size ? !(dec_ok && decode_integer_path(p)) : !pre_ok;
    Params q;
    int keep8 = 0;
    if (slow && path != (decode_size ? UNIQL_PATH_PREFILL : UNIQL_PATH_DECODE) && (keep8 = relay_candidate(p, &q)) != 0 &&
        (decode_size ? (decode_supported(q) && decode_integer_path(q)) : prefill_supported(q))) {
      if (!cfg.workspace) {
        int rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
        if (rc != UNIQL_OK) return rc;
      }
      const size_t bytes = (((size_t)p.M * (size_t)q.ldx * 2) + 255) & ~(size_t)255;
      const size_t floor_bytes = decode_size ? decode_workspace_bytes(p.M, p.K, 1) : decode_workspace_header_bytes();
      if (cfg.ws_bytes >= bytes + floor_bytes + 256) {
        // the copy lives at the end of the workspace; the kernels get what lies before it
        const size_t off = (cfg.ws_bytes - bytes) & ~(size_t)255;
        void* xr = reinterpret_cast<unsigned char*>(cfg.workspace) + off;
        const Fam& a = p.imap.fam[0];
        int rc = launch_relay_x(p.x, p.ldx, p.M, a.count, a.keep, keep8, xr, cfg.stream);
        if (rc != UNIQL_OK) return rc;
        q.x = xr;
        p = q;
        relaid = true;
        cfg.ws_bytes = off;
        dec_ok = p.M <= 16 && decode_supported(p);
        pre_ok = prefill_supported(p);
      }
    }
  }
  if (gv_else && !relaid) gv = true;
  if (path == UNIQL_PATH_AUTO)
    path = gv ? UNIQL_PATH_GEMV : dec_ok ? UNIQL_PATH_DECODE : (pre_ok ? UNIQL_PATH_PREFILL : UNIQL_PATH_GENERIC);
  if (path == UNIQL_PATH_GEMV) {
    if (!gemv_supported(p)) return UNIQL_ERR_UNSUPPORTED;
    if (!cfg.workspace) {
      int rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
      if (rc != UNIQL_OK) return rc;
    }
    return launch_gemv(p, cfg);
  }
  if (path == UNIQL_PATH_DECODE) {
    if (!(p.M <= 16 && decode_supported(p))) return UNIQL_ERR_UNSUPPORTED;
    if (!cfg.workspace) {
      int rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
      if (rc != UNIQL_OK) return rc;
    }
    // Batches of 9..16: the staged activations of 16 rows do not fit beside the stage ring, which would
    // force the input channels to be split over two groups of blocks and every tile through a hand-over.
    // The integer path streams the activations through the ring instead (one launch, the weights read once);
    // elsewhere two launches over half the batch each re-read the weights but still run more than twice as fast
    // as the split channels (option "decode_split_batch": 2 as described, 1 always two launches, 0 always one
    // launch with staged activations).
    const int sb = opt(kOptDecodeSplitBatch);
    const bool split_batch = sb == 1 || (sb == 2 && !decode_streams_batch(p));
    if (p.M > 8 && split_batch) {
      const int m1 = (p.M + 1) / 2;
      const size_t esz = 2;                               // fp16 / bf16
      Params a = p, b = p;
      a.M = m1;
      b.M = p.M - m1;
      b.x = reinterpret_cast<const unsigned char*>(p.x) + (size_t)m1 * p.ldx * esz;
      b.pos = p.pos ? p.pos + m1 : nullptr;
      for (int j = 0; j < p.n_jobs; ++j)
        b.job[j].y = reinterpret_cast<unsigned char*>(p.job[j].y) + (size_t)m1 * p.job[j].ldy * esz;
      int rc = launch_decode(a, cfg);
      if (rc != UNIQL_OK) return rc;
      return launch_decode(b, cfg);
    }
    return launch_decode(p, cfg);
  }
  if (path == UNIQL_PATH_PREFILL) {
    if (!prefill_supported(p)) return UNIQL_ERR_UNSUPPORTED;
    if (!cfg.workspace) {      // only the status word of the workspace is used
      int rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
      if (rc != UNIQL_OK) return rc;
    }
    return launch_prefill(p, cfg);
  }
  return launch_generic(p, cfg);
}

}  // namespace

int uniql::opt(int id) { return g_opt[id].load(std::memory_order_relaxed); }

extern "C" int uniql_set_option(const char* name, int value) {
  if (!name) return UNIQL_ERR_NULL;
  for (int i = 0; i < kOptCount; ++i)
    if (strcmp(name, kOpts[i].name) == 0) { g_opt[i].store(value); return UNIQL_OK; }
  return UNIQL_ERR_SHAPE;
}

extern "C" int uniql_version(void) { return 100; }

extern "C" const char* uniql_status_string(int s) {
  switch (s) {
    case UNIQL_OK: return "ok";
    case UNIQL_ERR_NULL: return "null pointer";
    case UNIQL_ERR_SHAPE: return "bad shape";
    case UNIQL_ERR_ALIGN: return "bad alignment";
    case UNIQL_ERR_DTYPE: return "bad dtype";
    case UNIQL_ERR_UNSUPPORTED: return "unsupported on the forced path";
    case UNIQL_ERR_WORKSPACE: return "workspace too small";
    case UNIQL_ERR_TIMEOUT: return "device-side wait timed out";
    case UNIQL_ERR_CUDA: return "CUDA error";
    default: return "unknown status";
  }
}

extern "C" int uniql_set_path(int path) {
  if (path < UNIQL_PATH_AUTO || path > UNIQL_PATH_GEMV) return UNIQL_ERR_SHAPE;
  g_path.store(path);
  return UNIQL_OK;
}

extern "C" size_t uniql_workspace_bytes(int M, int K, int N_total) {
  if (M < 1 || K < 1 || N_total < 1) return 0;
  // (+ room for the activations re-laid on 8-channel boundaries, see dispatch())
  const size_t relay = (((size_t)M * (size_t)(K + 8) * 2) + 255) / 256 * 256 + 512;
  if (M > 16) return prefill_workspace_bytes(M, K) + relay;
  const size_t a = decode_workspace_bytes(M, K, N_total), b = M <= 4 ? gemv_workspace_bytes(M, K, N_total) : 0;
  return (a > b ? a : b) + relay;
}

extern "C" int uniql_workspace_init(void* workspace, size_t bytes, void* stream) {
  if (!workspace) return UNIQL_ERR_NULL;
  if (((uintptr_t)workspace) & 255) return UNIQL_ERR_ALIGN;
  if (bytes == 0) return UNIQL_ERR_WORKSPACE;
  return cudaMemsetAsync(workspace, 0, bytes, (cudaStream_t)stream) == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

extern "C" int uniql_workspace_status(void* workspace, int* status) {
  if (!status) return UNIQL_ERR_NULL;
  if (!workspace) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return UNIQL_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_ws_mutex);
    workspace = g_ws[dev];
    if (!workspace) { *status = UNIQL_OK; return UNIQL_OK; }   // never used: nothing can have failed
  }
  int v = 0;
  if (cudaMemcpy(&v, reinterpret_cast<unsigned char*>(workspace) + decode_status_offset(), sizeof(int),
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return UNIQL_ERR_CUDA;
  *status = v;
  return UNIQL_OK;
}

extern "C" int uniql_qlinear_multi(const void* x, int ldx, int dt, int M, int K, const uniql_chanmap* in_map,
                                   int k_in, int n_jobs, const uniql_job* jobs, void* workspace,
                                   size_t ws_bytes, void* stream) {
  int rc = check_common(x, ldx, dt, M, K);
  if (rc) return rc;
  if (!jobs) return UNIQL_ERR_NULL;
  if (n_jobs < 1 || n_jobs > kMaxJobs) return UNIQL_ERR_SHAPE;
  if (workspace && (((uintptr_t)workspace) & 255)) return UNIQL_ERR_ALIGN;
  Params p;
  memset(&p, 0, sizeof(p));
  rc = compile_map(in_map, k_in, K, &p.imap);
  if (rc) return rc;
  p.x = x; p.ldx = ldx; p.dt = dt; p.M = M; p.K = K; p.k_in = p.imap.total;
  if (ldx < p.k_in) return UNIQL_ERR_SHAPE;
  p.n_jobs = n_jobs;
  for (int j = 0; j < n_jobs; ++j) {
    const uniql_job& s = jobs[j];
    rc = check_weight(s.packed_w, s.scales, s.zeros, s.N);
    if (rc) return rc;
    if (!s.y) return UNIQL_ERR_NULL;
    if ((((uintptr_t)s.y) & 1) || (s.bias && (((uintptr_t)s.bias) & 1))) return UNIQL_ERR_ALIGN;
    JobDev& d = p.job[j];
    rc = compile_map(s.out_map, s.k_out, s.N, &d.omap);
    if (rc) return rc;
    d.w = s.packed_w; d.scales = (const __half*)s.scales; d.zeros = (const __half*)s.zeros;
    d.bias = s.bias; d.y = s.y; d.ldy = s.ldy; d.N = s.N; d.k_out = d.omap.total;
    if (s.ldy < d.k_out) return UNIQL_ERR_SHAPE;
  }
  return dispatch(p, workspace, ws_bytes, stream);
}

extern "C" int uniql_qlinear_ex(const void* x, int ldx, int dt, const uint8_t* packed_w, const void* scales,
                                const void* zeros, const void* bias, int M, int K, int N,
                                const uniql_chanmap* in_map, int k_in, const uniql_chanmap* out_map,
                                int k_out, void* y, int ldy, void* workspace, size_t ws_bytes, void* stream) {
  uniql_job job;
  memset(&job, 0, sizeof(job));
  job.packed_w = packed_w; job.scales = scales; job.zeros = zeros; job.bias = bias;
  job.N = N; job.k_out = k_out; job.out_map = out_map; job.y = y; job.ldy = ldy;
  return uniql_qlinear_multi(x, ldx, dt, M, K, in_map, k_in, 1, &job, workspace, ws_bytes, stream);
}

extern "C" int uniql_qlinear(const void* x, const uint8_t* packed_w, const void* scales, const void* zeros,
                             int M, int K, int N, int k_in, int k_out, void* y, void* stream) {
  return uniql_qlinear_ex(x, k_in, UNIQL_F16, packed_w, scales, zeros, nullptr, M, K, N, nullptr, k_in,
                          nullptr, k_out, y, k_out, nullptr, 0, stream);
}

namespace {

// Q and K projections with the rotary epilogue and, when wv is given, the V projection (plain rows, the
// leading v_keep of every key-value head) as a third job of the same launch.
int qkv_rope_impl(const void* x, int ldx, int dt, const uint8_t* wq, const void* sq, const void* zq,
                  const uint8_t* wk, const void* sk, const void* zk, const uint8_t* wv, const void* sv,
                  const void* zv, const void* bq, const void* bk, const void* bv, int M, int K, int n_q_heads,
                  int n_kv_heads, int head_dim, int head_keep, int v_keep, const int32_t* retained_idx,
                  const int32_t* pos, double theta, const double* inv_freq, void* q_out, int ldq, void* k_out,
                  int ldk, void* v_out, int ldv, void* workspace, size_t ws_bytes, void* stream) {
  int rc = check_common(x, ldx, dt, M, K);
  if (rc) return rc;
  if (!retained_idx || !pos || !q_out || !k_out) return UNIQL_ERR_NULL;
  if (n_q_heads < 1 || n_kv_heads < 1 || (n_q_heads % n_kv_heads) != 0) return UNIQL_ERR_SHAPE;
  if (head_dim < 2 || (head_dim & 1) || head_dim > 2 * kMaxHalfDim) return UNIQL_ERR_SHAPE;
  if (head_keep < 2 || (head_keep & 1) || head_keep > head_dim) return UNIQL_ERR_SHAPE;
  if (!inv_freq && !(theta > 0.0)) return UNIQL_ERR_SHAPE;
  if (ldx < K) return UNIQL_ERR_SHAPE;   // the hidden dimension D_h is never pruned (Section 3.4)
  if (ldq < n_q_heads * head_keep || ldk < n_kv_heads * head_keep) return UNIQL_ERR_SHAPE;
  if ((((uintptr_t)q_out) & 1) || (((uintptr_t)k_out) & 1) || (((uintptr_t)retained_idx) & 3) ||
      (((uintptr_t)pos) & 3))
    return UNIQL_ERR_ALIGN;
  if ((bq && (((uintptr_t)bq) & 1)) || (bk && (((uintptr_t)bk) & 1))) return UNIQL_ERR_ALIGN;
  if (workspace && (((uintptr_t)workspace) & 255)) return UNIQL_ERR_ALIGN;
  rc = check_weight(wq, sq, zq, n_q_heads * head_dim);
  if (rc) return rc;
  rc = check_weight(wk, sk, zk, n_kv_heads * head_dim);
  if (rc) return rc;
  if (wv) {
    if (!v_out) return UNIQL_ERR_NULL;
    if (v_keep < 1 || v_keep > head_dim || ldv < n_kv_heads * v_keep) return UNIQL_ERR_SHAPE;
    if ((((uintptr_t)v_out) & 1) || (bv && (((uintptr_t)bv) & 1))) return UNIQL_ERR_ALIGN;
    rc = check_weight(wv, sv, zv, n_kv_heads * head_dim);
    if (rc) return rc;
  }

  Params p;
  memset(&p, 0, sizeof(p));
  compile_map(nullptr, K, K, &p.imap);
  p.x = x; p.ldx = ldx; p.dt = dt; p.M = M; p.K = K; p.k_in = K;
  p.n_jobs = wv ? 3 : 2;
  p.idx = retained_idx; p.pos = pos;
  for (int i = 0; i < head_dim / 2; ++i)
    p.rope_turn[i] = rope_turn_of(inv_freq ? inv_freq[i] : pow(theta, -2.0 * (double)i / (double)head_dim));
  for (int j = 0; j < 2; ++j) {
    JobDev& d = p.job[j];
    int nh = j == 0 ? n_q_heads : n_kv_heads;
    d.w = j == 0 ? wq : wk;
    d.scales = (const __half*)(j == 0 ? sq : sk);
    d.zeros = (const __half*)(j == 0 ? zq : zk);
    d.bias = j == 0 ? bq : bk;
    d.y = j == 0 ? q_out : k_out;
    d.ldy = j == 0 ? ldq : ldk;
    d.N = nh * head_dim;
    d.k_out = nh * head_keep;
    uniql_chanmap hm;
    hm.n_fam = 1;
    hm.fam[0] = uniql_family{0, head_dim / 2, head_keep / 2, 2 * nh};
    compile_map(&hm, 0, d.N, &d.omap);
    d.rope = RopeDesc{1, nh, j == 0 ? n_q_heads / n_kv_heads : 1, head_dim, head_keep};
  }
  if (wv) {
    JobDev& d = p.job[2];
    d.w = wv; d.scales = (const __half*)sv; d.zeros = (const __half*)zv; d.bias = bv;
    d.y = v_out; d.ldy = ldv; d.N = n_kv_heads * head_dim;
    uniql_chanmap hm;
    hm.n_fam = 1;
    hm.fam[0] = uniql_family{0, head_dim, v_keep, n_kv_heads};
    rc = compile_map(&hm, 0, d.N, &d.omap);
    if (rc) return rc;
    d.k_out = d.omap.total;
  }
  return dispatch(p, workspace, ws_bytes, stream);
}

}  // namespace

extern "C" int uniql_qk_rope_proj(const void* x, int ldx, int dt, const uint8_t* wq, const void* sq,
                                  const void* zq, const uint8_t* wk, const void* sk, const void* zk,
                                  const void* bq, const void* bk, int M, int K, int n_q_heads,
                                  int n_kv_heads, int head_dim, int head_keep, const int32_t* retained_idx,
                                  const int32_t* pos, double theta, const double* inv_freq, void* q_out,
                                  int ldq, void* k_out, int ldk, void* workspace, size_t ws_bytes,
                                  void* stream) {
  return qkv_rope_impl(x, ldx, dt, wq, sq, zq, wk, sk, zk, nullptr, nullptr, nullptr, bq, bk, nullptr, M, K,
                       n_q_heads, n_kv_heads, head_dim, head_keep, 0, retained_idx, pos, theta, inv_freq, q_out,
                       ldq, k_out, ldk, nullptr, 0, workspace, ws_bytes, stream);
}

extern "C" int uniql_qkv_rope_proj(const void* x, int ldx, int dt, const uint8_t* wq, const void* sq,
                                   const void* zq, const uint8_t* wk, const void* sk, const void* zk,
                                   const uint8_t* wv, const void* sv, const void* zv, const void* bq,
                                   const void* bk, const void* bv, int M, int K, int n_q_heads, int n_kv_heads,
                                   int head_dim, int head_keep, int v_keep, const int32_t* retained_idx,
                                   const int32_t* pos, double theta, const double* inv_freq, void* q_out,
                                   int ldq, void* k_out, int ldk, void* v_out, int ldv, void* workspace,
                                   size_t ws_bytes, void* stream) {
  if (!wv) return UNIQL_ERR_NULL;
  return qkv_rope_impl(x, ldx, dt, wq, sq, zq, wk, sk, zk, wv, sv, zv, bq, bk, bv, M, K, n_q_heads, n_kv_heads,
                       head_dim, head_keep, v_keep, retained_idx, pos, theta, inv_freq, q_out, ldq, k_out, ldk,
                       v_out, ldv, workspace, ws_bytes, stream);
}

namespace {

// SwiGLU MLP on the tensor-core kernel, two launches.  The first takes gate and up as a pair (their retained
// rows interleaved in every tile) and writes h = silu(x Wg^T) * (x Wu^T); the second is the plain down
// projection over the leading k_int channels of h.
int mlp_tensor_core(const void* x, int ldx, int dt, const uint8_t* wg, const void* sg, const void* zg, const uint8_t* wu,
                    const void* su, const void* zu, const uint8_t* wd, const void* sd, const void* zd, int M, int hidden,
                    int inter, int k_int, void* h, int ldh, void* y, int ldy, const LaunchCfg& cfg) {
  if ((hidden % kGroup) != 0 || (inter % kGroup) != 0) return UNIQL_ERR_SHAPE;
  Params a;
  memset(&a, 0, sizeof(a));
  compile_map(nullptr, hidden, hidden, &a.imap);
  a.x = x; a.ldx = ldx; a.dt = dt; a.M = M; a.K = hidden; a.k_in = hidden;
  a.n_jobs = 2;
  for (int j = 0; j < 2; ++j) {
    JobDev& jd = a.job[j];
    compile_map(nullptr, k_int, inter, &jd.omap);
    jd.w = j == 0 ? wg : wu;
    jd.scales = (const __half*)(j == 0 ? sg : su);
    jd.zeros = (const __half*)(j == 0 ? zg : zu);
    jd.y = h; jd.ldy = ldh; jd.N = inter; jd.k_out = k_int;
    jd.pair = j + 1;
  }
  if (!prefill_supported(a)) return UNIQL_ERR_UNSUPPORTED;
  int rc = launch_prefill(a, cfg);
  if (rc != UNIQL_OK) return rc;
  Params b;
  memset(&b, 0, sizeof(b));
  compile_map(nullptr, k_int, inter, &b.imap);
  b.x = h; b.ldx = ldh; b.dt = dt; b.M = M; b.K = inter; b.k_in = k_int;
  b.n_jobs = 1;
  JobDev& jd = b.job[0];
  compile_map(nullptr, hidden, hidden, &jd.omap);
  jd.w = wd; jd.scales = (const __half*)sd; jd.zeros = (const __half*)zd;
  jd.y = y; jd.ldy = ldy; jd.N = hidden; jd.k_out = hidden;
  return dispatch(b, cfg.workspace, cfg.ws_bytes, cfg.stream);
}

}  // namespace

extern "C" size_t uniql_mlp_workspace_bytes(int M, int hidden, int inter) {
  if (M < 1 || hidden < 1 || inter < 1) return 0;
  if (M > 16) return prefill_workspace_bytes(M, hidden > inter ? hidden : inter);     // tensor-core kernel, two launches
  // (16 rows or fewer in bf16 also run on the tensor-core kernel: room for its fp16 copy of the activations)
  const size_t a = mlp_decode_workspace_bytes(M, hidden, inter), b = prefill_workspace_bytes(M, hidden > inter ? hidden : inter);
  size_t c = 0;
  if (M <= 4) {
    const size_t c0 = gemv_workspace_bytes(M, hidden, 2 * inter), c1 = gemv_workspace_bytes(M, inter, hidden);
    c = c0 > c1 ? c0 : c1;
  }
  return a > b ? (a > c ? a : c) : (b > c ? b : c);
}

extern "C" int uniql_mlp_swiglu_decode(const void* x, int ldx, const uint8_t* wg, const void* sg, const void* zg,
                                       const uint8_t* wu, const void* su, const void* zu, const uint8_t* wd,
                                       const void* sd, const void* zd, int M, int hidden, int inter, int k_int,
                                       void* h, int ldh, void* y, int ldy, int fuse, void* workspace,
                                       size_t ws_bytes, void* stream) {
  if (!x || !h || !y) return UNIQL_ERR_NULL;
  if (M < 1 || hidden < kGroup || inter < kGroup || k_int < 1 || k_int > inter) return UNIQL_ERR_SHAPE;
  if (ldx < hidden || ldh < k_int || ldy < hidden) return UNIQL_ERR_SHAPE;
  if (fuse < -1 || fuse > 1) return UNIQL_ERR_SHAPE;
  int rc = check_weight(wg, sg, zg, inter);
  if (!rc) rc = check_weight(wu, su, zu, inter);
  if (!rc) rc = check_weight(wd, sd, zd, hidden);
  if (rc) return rc;
  if ((((uintptr_t)x) | ((uintptr_t)h) | ((uintptr_t)y)) & 1) return UNIQL_ERR_ALIGN;
  if (workspace && (((uintptr_t)workspace) & 255)) return UNIQL_ERR_ALIGN;
  if (cudaPeekAtLastError() != cudaSuccess) return UNIQL_ERR_CUDA;
  LaunchCfg cfg{workspace, ws_bytes, (cudaStream_t)stream};
  if (!cfg.workspace) {
    rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
    if (rc != UNIQL_OK) return rc;
  }
  if (M > 16) {
    if (fuse == 1) return UNIQL_ERR_UNSUPPORTED;
    return mlp_tensor_core(x, ldx, UNIQL_F16, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, ldh, y, ldy, cfg);
  }
  MlpDecode d;
  memset(&d, 0, sizeof(d));
  d.x = x; d.ldx = ldx; d.M = M; d.hidden = hidden; d.inter = inter; d.k_int = k_int;
  d.wg = wg; d.wu = wu; d.wd = wd;
  d.sg = (const __half*)sg; d.zg = (const __half*)zg; d.su = (const __half*)su; d.zu = (const __half*)zu;
  d.sd = (const __half*)sd; d.zd = (const __half*)zd;
  d.h = h; d.ldh = ldh; d.y = y; d.ldy = ldy;
  // one to four rows: two launches of the streaming kernel (unless one launch or the persistent kernel is asked for)
  if (fuse != 1 && gemv_mlp_supported(d) &&
      (g_path.load() == UNIQL_PATH_GEMV ||
       (g_path.load() == UNIQL_PATH_AUTO && (opt(kOptGemvFirst) == 1 || !mlp_decode_supported(d)))))
    return launch_gemv_mlp(d, cfg);
  if (g_path.load() == UNIQL_PATH_GEMV) return UNIQL_ERR_UNSUPPORTED;
  if (!mlp_decode_supported(d)) return UNIQL_ERR_UNSUPPORTED;
  auto run = [&](const MlpDecode& q) -> int {
    // fuse = -1 takes two launches: on B200 the launch boundary (programmatic dependent launch) costs less
    // than the grid-wide barrier of the single launch (measured 29.2 us against 32.6 us per Llama-3-8B layer)
    return launch_mlp_decode(q, fuse == 1 ? 1 : 0, cfg);
  };
  // (nine to sixteen rows: one pass with streamed activations, or under option "decode_split_batch" 0 / 1 as for
  // the plain decode path)
  if (M > 8 && fuse != 1 && !(opt(kOptDecodeSplitBatch) == 2 && opt(kOptDecodeXstream) != 0 && opt(kOptDecodeI8) != 0)) {
    const int m1 = (M + 1) / 2;
    MlpDecode a = d, b = d;
    a.M = m1;
    b.M = M - m1;
    b.x = reinterpret_cast<const unsigned char*>(x) + (size_t)m1 * ldx * 2;
    b.h = reinterpret_cast<unsigned char*>(h) + (size_t)m1 * ldh * 2;
    b.y = reinterpret_cast<unsigned char*>(y) + (size_t)m1 * ldy * 2;
    if (!mlp_decode_supported(b)) return UNIQL_ERR_UNSUPPORTED;
    rc = run(a);
    return rc ? rc : run(b);
  }
  return run(d);
}

extern "C" int uniql_mlp_swiglu(const void* x, int ldx, int dt, const uint8_t* wg, const void* sg, const void* zg,
                                const uint8_t* wu, const void* su, const void* zu, const uint8_t* wd, const void* sd,
                                const void* zd, int M, int hidden, int inter, int k_int, void* h, int ldh, void* y,
                                int ldy, void* workspace, size_t ws_bytes, void* stream) {
  if (dt != UNIQL_F16 && dt != UNIQL_BF16) return UNIQL_ERR_DTYPE;
  if (dt == UNIQL_F16 && M <= 16)
    return uniql_mlp_swiglu_decode(x, ldx, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, ldh, y, ldy,
                                   -1, workspace, ws_bytes, stream);
  if (!x || !h || !y) return UNIQL_ERR_NULL;
  if (M < 1 || hidden < kGroup || inter < kGroup || k_int < 1 || k_int > inter) return UNIQL_ERR_SHAPE;
  if (ldx < hidden || ldh < k_int || ldy < hidden) return UNIQL_ERR_SHAPE;
  int rc = check_weight(wg, sg, zg, inter);
  if (!rc) rc = check_weight(wu, su, zu, inter);
  if (!rc) rc = check_weight(wd, sd, zd, hidden);
  if (rc) return rc;
  if ((((uintptr_t)x) | ((uintptr_t)h) | ((uintptr_t)y)) & 1) return UNIQL_ERR_ALIGN;
  if (workspace && (((uintptr_t)workspace) & 255)) return UNIQL_ERR_ALIGN;
  if (cudaPeekAtLastError() != cudaSuccess) return UNIQL_ERR_CUDA;
  LaunchCfg cfg{workspace, ws_bytes, (cudaStream_t)stream};
  if (!cfg.workspace) {
    rc = lib_workspace(&cfg.workspace, &cfg.ws_bytes, cfg.stream);
    if (rc != UNIQL_OK) return rc;
  }
  return mlp_tensor_core(x, ldx, dt, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, ldh, y, ldy, cfg);
}
