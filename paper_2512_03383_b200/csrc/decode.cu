// Decode kernel (M = 1..16) of the pruned 4-bit linear layer, sm_100a.
//
// The decode step streams every retained weight once (weight-bandwidth bound), so the kernel is
// organised around 128-bit loads of packed codes straight from the interchange layout: lane (r, c)
// of a warp loads the 32 codes c*32..c*32+31 of one 128-channel quantisation group for weight rows
// r and r+8 of a 16-row tile, i.e. exactly the A fragments of eight m16n8k16 tensor-core MMAs whose
// B fragments are the (permuted) activations.  The contraction index of an MMA is only a label, so
// the activations are staged in shared memory in the order the nibbles come out of a 32-bit word
// and no weight byte is ever shuffled.  The MMAs run on the integer codes (code-8 is exact in
// fp16/bf16); scale and zero-point are applied once per group and row in fp32:
//   y += s * (sum_k (q_k-8) x_k  -  (z-8) * sum_k x_k),
// which makes the result independent of the activation dtype's mantissa.
// Truncation to the leading sorted channels (Section 3.4) is pure index arithmetic: pruned rows are
// never addressed, pruned input channels are either outside the visited groups or meet a zero
// activation.
// Scheduling: one persistent block of 16 warps per SM.  All (row tile, k-chunk) units of the launch
// form one k-fastest sequence that is cut into equal contiguous ranges, one per warp (stream-K), so
// every SM streams the same number of bytes and nothing is launched in waves.  A warp keeps the loads
// of its next chunk in flight while it works on the current one, accumulates in registers while it
// stays on a tile, and when it leaves a tile that other warps also worked on it parks its partial sum
// in a workspace slot; the last warp to arrive adds the slots in a fixed order (deterministic, no
// spinning).  When the activations of a block do not fit in shared memory (large M x K) the input
// channels are split into k-parts with their own blocks.
// The rotary epilogue (Section 3.2, fused RoPE) needs both members of a rotation pair: in rope mode
// a 16-row tile is 8 pairs, first-half members in rows 0..7 and their partners in rows 8..15, which
// is exactly the (r, r+8) row pair a lane owns in the MMA accumulator layout.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace uniql {
namespace {

constexpr int NW = 16;            // warps per block
constexpr int NTD = NW * 32;      // threads per block
constexpr int kMaxSpans = kMaxFam;
constexpr int kCounterInts = 1 << 16;   // arrival counters (one per row tile) at the head of the workspace
constexpr int kMaxKParts = 16;
constexpr size_t kSmemBudget = 200 * 1024;

struct DecodeCfg {
  int n_kp, n_rp;        // k-parts x row-parts = blocks
  int gp;                // visited groups per k-part (the last part may be shorter)
  int tiles_total;
  int tile_begin[kMaxJobs + 1];   // first global tile of each job
  int row_base[kMaxJobs];         // (unused by the kernel; kept for sizing)
  int g_total;           // visited 128-channel groups
  int n_spans;
  int vg_begin[kMaxSpans + 1];  // visit index at which span s starts
  int vg_first[kMaxSpans];      // its first stored group
  int x_vec;             // activations can be staged with 128-bit loads
  int sz_vec;            // scales / zero-points of a chunk can be fetched with one vector load
  int mp;                // activation rows staged in shared memory
  int max_slots;         // workspace slots per tile
  int* counters;
  float* partials;
};

__device__ inline int visit_to_group(const DecodeCfg& c, int v) {
  int s = 0;
  while (s + 1 < c.n_spans && v >= c.vg_begin[s + 1]) ++s;
  return c.vg_first[s] + (v - c.vg_begin[s]);
}

__device__ inline uint4 ldg_stream(const void* ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr));
  return v;
}
__device__ inline uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ inline float2 lds64f(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

// (a & mask) | magic in one LOP3 (truth table 0xEA)
__device__ inline uint32_t and_or(uint32_t a, uint32_t mask, uint32_t magic) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(magic));
  return d;
}

template <typename T> struct Cvt;
// fp16: a nibble in bits [3:0] of a 16-bit half ORed onto 0x6400 reads 1024+q, one in bits [7:4]
// ORed onto 0x5400 reads 64+q; subtracting 1032 / 72 leaves q-8 exactly.
template <> struct Cvt<__half> {
  static __device__ inline void word(uint32_t w, uint32_t (&a)[4]) {
    const uint32_t k_lo = 0x64086408u, k_hi = 0x54805480u;   // 1032, 72
    const uint32_t w8 = w >> 8;
    const uint32_t t0 = and_or(w, 0x000f000fu, 0x64006400u);
    const uint32_t t1 = and_or(w, 0x00f000f0u, 0x54005400u);
    const uint32_t t2 = and_or(w8, 0x000f000fu, 0x64006400u);
    const uint32_t t3 = and_or(w8, 0x00f000f0u, 0x54005400u);
    asm("sub.f16x2 %0, %1, %2;" : "=r"(a[0]) : "r"(t0), "r"(k_lo));
    asm("sub.f16x2 %0, %1, %2;" : "=r"(a[1]) : "r"(t1), "r"(k_hi));
    asm("sub.f16x2 %0, %1, %2;" : "=r"(a[2]) : "r"(t2), "r"(k_lo));
    asm("sub.f16x2 %0, %1, %2;" : "=r"(a[3]) : "r"(t3), "r"(k_hi));
  }
  static __device__ inline void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                    uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
  static __device__ inline void mma0(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                     uint32_t b0, uint32_t b1) {   // d = a*b (zero accumulator input)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
  }
};
// bf16 has 7 mantissa bits: only a nibble in bits [3:0] can be ORed onto 0x4300 (128+q).
template <> struct Cvt<__nv_bfloat16> {
  static __device__ inline void word(uint32_t w, uint32_t (&a)[4]) {
    const uint32_t k136 = 0x43084308u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t t = and_or(w >> (4 * i), 0x000f000fu, 0x43004300u);
      asm("sub.bf16x2 %0, %1, %2;" : "=r"(a[i]) : "r"(t), "r"(k136));
    }
  }
  static __device__ inline void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                    uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
  static __device__ inline void mma0(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                     uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
  }
};

// The two weight rows a lane owns in a 16-row tile.
struct LaneRows {
  int sr0, sr1;      // stored rows (clamped to a valid row when the slot is empty)
  int oc0, oc1;      // compact output columns, -1 when empty
  int rope_p, rope_kvh;
};

__device__ inline LaneRows resolve_rows(const JobDev& jb, int tile, int r) {
  LaneRows L;
  L.rope_p = 0; L.rope_kvh = 0;
  if (jb.rope.enabled) {
    const int half = jb.rope.head_keep >> 1;
    const int P = tile * 8 + r;
    const bool ok = P < jb.rope.n_heads * half;
    const int Pc = ok ? P : 0;
    const int h = Pc / half, cc = Pc - h * half;
    L.sr0 = h * jb.rope.head_dim + cc;
    L.sr1 = L.sr0 + (jb.rope.head_dim >> 1);
    L.oc0 = ok ? h * jb.rope.head_keep + cc : -1;
    L.oc1 = ok ? L.oc0 + half : -1;
    L.rope_p = cc;
    L.rope_kvh = h / jb.rope.rep;
  } else {
    const int j0 = tile * 16 + r, j1 = j0 + 8;
    L.oc0 = j0 < jb.k_out ? j0 : -1;
    L.oc1 = j1 < jb.k_out ? j1 : -1;
    if (jb.omap.n_fam == 1 && jb.omap.fam[0].count == 1) {
      L.sr0 = jb.omap.fam[0].start + (L.oc0 >= 0 ? j0 : 0);
      L.sr1 = jb.omap.fam[0].start + (L.oc1 >= 0 ? j1 : 0);
    } else {
      L.sr0 = map_compact_to_stored(jb.omap, L.oc0 >= 0 ? j0 : 0);
      L.sr1 = map_compact_to_stored(jb.omap, L.oc1 >= 0 ? j1 : 0);
    }
  }
  return L;
}

// bias, rotary embedding on the retained pair, one rounding, store
template <typename T, int MT>
__device__ inline void epilogue(const Params& p, const JobDev& jb, const LaneRows& L, int cq, float (&out)[MT][4]) {
  const T* bias = reinterpret_cast<const T*>(jb.bias);
  const float b0 = (bias && L.oc0 >= 0) ? DT<T>::to_f(bias[L.sr0]) : 0.f;
  const float b1 = (bias && L.oc1 >= 0) ? DT<T>::to_f(bias[L.sr1]) : 0.f;
  T* y = reinterpret_cast<T*>(jb.y);
  double invf = 0.0;
  if (jb.rope.enabled) {
    int pidx = p.idx[L.rope_kvh * (jb.rope.head_keep >> 1) + L.rope_p];
    pidx = min(max(pidx, 0), (jb.rope.head_dim >> 1) - 1);
    invf = p.inv_freq[pidx];
  }
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int m = 2 * cq + e + 8 * t;
      if (m >= p.M) continue;
      float lo = out[t][e] + b0, hi = out[t][2 + e] + b1;
      if (jb.rope.enabled) {
        float cs, sn;
        rope_cos_sin(p.pos[m], invf, cs, sn);
        const float a = lo, b = hi;
        lo = a * cs - b * sn;
        hi = b * cs + a * sn;
      }
      if (L.oc0 >= 0) y[(size_t)m * jb.ldy + L.oc0] = DT<T>::from_f(lo);
      if (L.oc1 >= 0) y[(size_t)m * jb.ldy + L.oc1] = DT<T>::from_f(hi);
    }
}

// ---------------------------------------------------------------------------------------- kernel
__device__ inline int owner_of(long u, long W, long U) {
  // the warp whose range [U*w/W, U*(w+1)/W) holds unit u; exact in fp64 for these magnitudes
  return (int)floor(((double)(u + 1) * (double)W - 1.0) / (double)U);
}

// A warp leaves tile `tgl`: finish it alone, or park the partial sum in its workspace slot and let the
// last warp to arrive add all slots in slot order and finish.  Kept out of line: it runs once or twice
// per warp and would only bloat the streaming loop.  Everything is passed by value so that the caller's
// accumulators stay in registers.
constexpr int MT_MAX = 2;
struct OutVals { float v[MT_MAX][4]; };
template <typename T, int MT, int CH>
__device__ __noinline__ void flush_tile(const Params& p, const DecodeCfg& c, int kp, int gw, int tgl, int jl,
                                        const LaneRows Ll, int lane, const OutVals ov) {
  const int r = lane >> 2, cq = lane & 3;
  float out[MT][4];
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) out[t][i] = ov.v[t][i];
  const long Wall = (long)c.n_rp * NW;
  int total = 0, my_slot = 0;
  for (int q = 0; q < c.n_kp; ++q) {
    const int Gq = min(c.gp, c.g_total - q * c.gp);
    const long Cq = (Gq + CH - 1) / CH;
    const long Uq = (long)c.tiles_total * Cq;
    const long Wq = Wall < Uq ? Wall : Uq;
    const int first = owner_of((long)tgl * Cq, Wq, Uq);
    const int last = owner_of((long)tgl * Cq + Cq - 1, Wq, Uq);
    if (q == kp) my_slot = total + (gw - first);
    total += last - first + 1;
  }
  if (total == 1) {
    epilogue<T, MT>(p, p.job[jl], Ll, cq, out);
    return;
  }
  const size_t slot_floats = (size_t)p.M * 16;
  float* tile_part = c.partials + (size_t)tgl * c.max_slots * slot_floats;
  float* mine = tile_part + (size_t)my_slot * slot_floats;
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int m = 2 * cq + e + 8 * t;
      if (m >= p.M) continue;
      __stcg(mine + m * 16 + r, out[t][e]);
      __stcg(mine + m * 16 + r + 8, out[t][2 + e]);
    }
  __threadfence();
  __syncwarp();
  int last_arrival = 0;
  if (lane == 0) last_arrival = atomicAdd(&c.counters[tgl], 1) == total - 1;
  last_arrival = __shfl_sync(0xffffffffu, last_arrival, 0);
  if (!last_arrival) return;
  __threadfence();
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) out[t][i] = 0.f;
  for (int s2 = 0; s2 < total; ++s2) {
    const float* src = tile_part + (size_t)s2 * slot_floats;
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int m = 2 * cq + e + 8 * t;
        if (m >= p.M) continue;
        out[t][e] += __ldcg(src + m * 16 + r);
        out[t][2 + e] += __ldcg(src + m * 16 + r + 8);
      }
  }
  epilogue<T, MT>(p, p.job[jl], Ll, cq, out);
  if (lane == 0) c.counters[tgl] = 0;       // ready for the next call
}

template <typename T, int MT, int CH>
__global__ void __launch_bounds__(NTD, 1) decode_kernel(const __grid_constant__ Params p,
                                                        const __grid_constant__ DecodeCfg c) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = lane >> 2, cq = lane & 3;
  const int mp = c.mp;
  const int kp = blockIdx.x / c.n_rp, rp = blockIdx.x - kp * c.n_rp;
  const int v_lo = kp * c.gp;                                   // first visit index of this k-part
  const int Gk = min(c.gp, c.g_total - v_lo);                   // its groups
  const int Ck = (Gk + CH - 1) / CH;                            // chunks per tile
  // shared memory: staged activations, mp rows + one all-zero row of (gp*256+64) bytes each (a group is
  // 256 bytes; the 64-byte pad puts the two rows met by one 128-bit load phase on distinct banks), then
  // the per-group activation sums [gp][8*MT] fp32
  const int row_bytes = c.gp * 256 + 64;
  const int xg_off = (mp + 1) * row_bytes;
  float* xg = reinterpret_cast<float*>(smem + xg_off);
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
  const int sg_lo = visit_to_group(c, v_lo);
  const bool contig = visit_to_group(c, v_lo + Gk - 1) == sg_lo + Gk - 1;   // block-uniform

  // ---- this warp's contiguous range of (tile, chunk) units, k fastest
  const long U = (long)c.tiles_total * Ck;
  const long Wall = (long)c.n_rp * NW;
  const long W = Wall < U ? Wall : U;                           // warps that get work
  const int gw = rp * NW + warp;
  int ub = 0, ue = 0;
  if (gw < W) { ub = (int)(U * gw / W); ue = (int)(U * (gw + 1) / W); }

  const int G = p.K / kGroup;
  auto job_of = [&](int tg) { int j = 0; while (j + 1 < p.n_jobs && tg >= c.tile_begin[j + 1]) ++j; return j; };

  // packed codes of the CH groups of the current chunk (reloaded in place, group by group, with the
  // next chunk's codes as soon as a group has been consumed) and fp16 scale / zero pairs
  uint4 w0[CH], w1[CH];
  uint32_t sc[4][CH / 2], scn[4][CH / 2];   // s(row r), z(row r), s(row r+8), z(row r+8); two groups per word

  auto load_group = [&](int g, const uint8_t* q0, const uint8_t* q1, int chn) {
    // q0/q1: row pointers already advanced to this lane's 16 bytes of stored group sg_lo (contiguous case)
    const int gi = chn * CH + g;
    if (gi < Gk) {
      const size_t off = (size_t)(contig ? sg_lo + gi : visit_to_group(c, v_lo + gi)) * 64;
      w0[g] = ldg_stream(q0 + off);
      w1[g] = ldg_stream(q1 + off);
    }
  };
  auto load_scales = [&](uint32_t (&dst)[4][CH / 2], const JobDev& jb, const LaneRows& L, int chn) {
    const int g0 = chn * CH;
    const __half* base[4] = {jb.scales + (size_t)L.sr0 * G, jb.zeros + (size_t)L.sr0 * G,
                             jb.scales + (size_t)L.sr1 * G, jb.zeros + (size_t)L.sr1 * G};
    if (c.sz_vec) {     // chunk start is CH-aligned in stored groups and the CH values are contiguous
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if constexpr (CH == 4) {
          const uint2 v = __ldg(reinterpret_cast<const uint2*>(base[q] + sg_lo + g0));
          dst[q][0] = v.x; dst[q][1] = v.y;
        } else {
          dst[q][0] = __ldg(reinterpret_cast<const uint32_t*>(base[q] + sg_lo + g0));
        }
      }
    } else {
      const int nv = min(CH, Gk - g0);
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int g = 0; g < CH; g += 2) {
          const int ga = visit_to_group(c, v_lo + g0 + (g < nv ? g : 0));
          const int gb = visit_to_group(c, v_lo + g0 + (g + 1 < nv ? g + 1 : 0));
          const uint32_t lo = __half_as_ushort(__ldg(base[q] + ga));
          const uint32_t hi = __half_as_ushort(__ldg(base[q] + gb));
          dst[q][g >> 1] = lo | (hi << 16);
        }
    }
  };

  // the first chunk's loads go out before the activations are staged (they do not depend on them)
  int tg = 0, ch = 0, jn = 0;
  LaneRows L;
  if (ub < ue) {
    tg = ub / Ck; ch = ub - tg * Ck;
    jn = job_of(tg);
    L = resolve_rows(p.job[jn], tg - c.tile_begin[jn], r);
    const uint8_t* q0 = p.job[jn].w + (size_t)L.sr0 * (p.K / 2) + cq * 16;
    const uint8_t* q1 = p.job[jn].w + (size_t)L.sr1 * (p.K / 2) + cq * 16;
#pragma unroll
    for (int g = 0; g < CH; ++g) load_group(g, q0, q1, ch);
    load_scales(sc, p.job[jn], L, ch);
  }

  // ---- stage activations: permuted into nibble order, zero where the channel is pruned
  {
    const T* x = reinterpret_cast<const T*>(p.x);
    uint4* xs = reinterpret_cast<uint4*>(smem);
    const int row_units = row_bytes / 16;
    for (int i = tid; i < row_units; i += NTD) xs[mp * row_units + i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < c.gp * 8 * MT; i += NTD) xg[i] = 0.f;
    __syncthreads();
    if (c.x_vec) {
      const int start = p.imap.fam[0].start, keep = p.imap.fam[0].keep;
      const int n_units = Gk * mp * 16;
      for (int u = tid; u < ((n_units + 31) & ~31); u += NTD) {   // whole warps stay in the shuffles
        const bool in_range = u < n_units;
        const int u16 = u & 15, pair = in_range ? u >> 4 : 0;
        const int m = pair / Gk, lv = pair - m * Gk;
        uint4 in = make_uint4(0, 0, 0, 0);
        if (in_range && m < p.M) {
          const int t0 = (contig ? sg_lo + lv : visit_to_group(c, v_lo + lv)) * kGroup + 8 * u16 - start;
          if (t0 >= 0 && t0 < keep) in = *reinterpret_cast<const uint4*>(x + (size_t)m * p.ldx + t0);
        }
        uint4 o;
        o.x = __byte_perm(in.x, in.z, 0x5410); o.y = __byte_perm(in.x, in.z, 0x7632);
        o.z = __byte_perm(in.y, in.w, 0x5410); o.w = __byte_perm(in.y, in.w, 0x7632);
        // unit (chunk c', word j) of a group sits at byte j*64 + c'*16; u16 = c'*4 + j
        if (in_range) xs[m * row_units + lv * 16 + (u16 & 3) * 4 + (u16 >> 2)] = o;
        const typename DT<T>::T2* h2 = reinterpret_cast<const typename DT<T>::T2*>(&in);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 f = DT<T>::to_f2(h2[i]); sum += f.x + f.y; }
#pragma unroll
        for (int o2 = 8; o2 >= 1; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
        if (in_range && u16 == 0) xg[lv * 8 * MT + m] = sum;
      }
    } else {
      T* xh = reinterpret_cast<T*>(smem);
      const int n_pairs = Gk * mp;
      for (int pair = warp; pair < n_pairs; pair += NW) {
        const int m = pair / Gk, lv = pair - m * Gk;
        const bool live = m < p.M;
        const int kbase = visit_to_group(c, v_lo + lv) * kGroup;
        float sum = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int i = lane + 32 * q;
          T val = DT<T>::from_f(0.f);
          if (live) {
            const int t = map_stored_to_compact(p.imap, kbase + i);
            if (t >= 0) val = x[(size_t)m * p.ldx + t];
          }
          const int ccq = i >> 5, j = (i & 31) >> 3, e = i & 7;
          xh[(m * row_units + lv * 16 + j * 4 + ccq) * 8 + 2 * (e & 3) + (e >> 2)] = val;
          sum += DT<T>::to_f(val);
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
        if (lane == 0) xg[lv * 8 * MT + m] = sum;
      }
    }
  }
  __syncthreads();
  if (ub >= ue) return;

  // per-lane shared-memory address of the B fragments (lanes beyond the staged rows read the zero row)
  uint32_t xb_addr[MT];
#pragma unroll
  for (int t = 0; t < MT; ++t) {
    const int m = r + 8 * t;
    xb_addr[t] = smem_base + (uint32_t)((m < mp ? m : mp) * row_bytes + cq * 16);
  }
  const uint32_t xg_addr = smem_base + (uint32_t)xg_off + (uint32_t)(2 * cq * 4);

  float out[MT][4];
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) out[t][i] = 0.f;

  // ---- stream the units: while group g of the current chunk is consumed, group g of the next chunk
  //      is already being fetched into the registers group g-1 has just freed
  for (int u = ub;; ++u) {
    const bool has_next = u + 1 < ue;
    int tg1 = tg, ch1 = ch + 1, jn1 = jn;
    LaneRows L1 = L;
    if (ch1 == Ck) { ch1 = 0; tg1 = tg + 1; }
    const uint8_t* q0 = nullptr;
    const uint8_t* q1 = nullptr;
    if (has_next) {
      if (tg1 != tg) {
        jn1 = job_of(tg1);
        L1 = resolve_rows(p.job[jn1], tg1 - c.tile_begin[jn1], r);
      }
      q0 = p.job[jn1].w + (size_t)L1.sr0 * (p.K / 2) + cq * 16;
      q1 = p.job[jn1].w + (size_t)L1.sr1 * (p.K / 2) + cq * 16;
      load_scales(scn, p.job[jn1], L1, ch1);
    }
    const int g0 = ch * CH;
    const int nvalid = min(CH, Gk - g0);
    uint32_t xa[MT];
#pragma unroll
    for (int t = 0; t < MT; ++t) xa[t] = xb_addr[t] + (uint32_t)(g0 * 256);
    const uint32_t xga = xg_addr + (uint32_t)(g0 * 8 * MT * 4);
#pragma unroll
    for (int g = 0; g < CH; ++g) {
      if (g < nvalid) {
        float acc[MT][2][4];     // two accumulators per batch tile: two independent MMA chains
        const uint32_t wa[4] = {w0[g].x, w0[g].y, w0[g].z, w0[g].w};
        const uint32_t wb[4] = {w1[g].x, w1[g].y, w1[g].z, w1[g].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t a[4], b[4];
          Cvt<T>::word(wa[j], a);
          Cvt<T>::word(wb[j], b);
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            const uint4 xb = lds128(xa[t] + (uint32_t)(g * 256 + j * 64));
            if (j == 0) {
              Cvt<T>::mma0(acc[t][0], a[0], b[0], a[1], b[1], xb.x, xb.y);
              Cvt<T>::mma0(acc[t][1], a[2], b[2], a[3], b[3], xb.z, xb.w);
            } else {
              Cvt<T>::mma(acc[t][0], a[0], b[0], a[1], b[1], xb.x, xb.y);
              Cvt<T>::mma(acc[t][1], a[2], b[2], a[3], b[3], xb.z, xb.w);
            }
          }
        }
        if (has_next) load_group(g, q0, q1, ch1);      // the registers of group g are free again
        auto pick = [&](int q) -> float {
          const __half2 h = *reinterpret_cast<const __half2*>(&sc[q][g >> 1]);
          return (g & 1) ? __high2float(h) : __low2float(h);
        };
        const float s0 = pick(0), nz0 = 8.f - pick(1);
        const float s1 = pick(2), nz1 = 8.f - pick(3);
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          const float2 X = lds64f(xga + (uint32_t)((g * 8 * MT + 8 * t) * 4));
          out[t][0] = fmaf(s0, fmaf(nz0, X.x, acc[t][0][0] + acc[t][1][0]), out[t][0]);
          out[t][1] = fmaf(s0, fmaf(nz0, X.y, acc[t][0][1] + acc[t][1][1]), out[t][1]);
          out[t][2] = fmaf(s1, fmaf(nz1, X.x, acc[t][0][2] + acc[t][1][2]), out[t][2]);
          out[t][3] = fmaf(s1, fmaf(nz1, X.y, acc[t][0][3] + acc[t][1][3]), out[t][3]);
        }
      } else if (has_next) {
        load_group(g, q0, q1, ch1);
      }
    }
    if (!has_next || tg1 != tg) {
      OutVals ov;
#pragma unroll
      for (int t = 0; t < MT_MAX; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) ov.v[t][i] = t < MT ? out[t < MT ? t : 0][i] : 0.f;
      flush_tile<T, MT, CH>(p, c, kp, gw, tg, jn, L, lane, ov);
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) out[t][i] = 0.f;
    }
    if (!has_next) break;
    tg = tg1; ch = ch1; jn = jn1; L = L1;
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int i = 0; i < CH / 2; ++i) sc[q][i] = scn[q][i];
  }
}

// -------------------------------------------------------------------------------- host side
int env_int(const char* name, int dflt) {
  const char* s = getenv(name);
  return s ? atoi(s) : dflt;
}

int job_tiles(const JobDev& j) {
  if (j.rope.enabled) return (j.rope.n_heads * (j.rope.head_keep / 2) + 7) / 8;
  return (j.k_out + 15) / 16;
}

// Visited-group spans of the input map: every 128-channel group that holds a retained channel,
// neighbouring families merged when they touch the same group.
void build_spans(const ChanMap& m, DecodeCfg* c) {
  int n = 0, total = 0;
  int last_g = -1;
  for (int f = 0; f < m.n_fam; ++f) {
    const Fam& a = m.fam[f];
    int first = a.start / kGroup;
    int end = a.start + (a.count - 1) * a.period + a.keep;   // exclusive
    int last = (end - 1) / kGroup;
    if (n > 0 && first <= last_g) {
      if (last > last_g) { total += last - last_g; last_g = last; }
    } else {
      c->vg_begin[n] = total;
      c->vg_first[n] = first;
      total += last - first + 1;
      last_g = last;
      ++n;
    }
  }
  c->n_spans = n;
  c->vg_begin[n] = total;
  c->g_total = total;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      n = 148;
  }
  return n;
}

size_t smem_bytes(int mp, int gp, int MT) { return (size_t)(mp + 1) * (gp * 256 + 64) + (size_t)gp * 8 * MT * 4; }

template <typename T, int MT, int CH>
int launch_t(const Params& p, const DecodeCfg& c, cudaStream_t stream) {
  const size_t smem = smem_bytes(c.mp, c.gp, MT);
  auto kern = decode_kernel<T, MT, CH>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return UNIQL_ERR_CUDA;
  kern<<<c.n_kp * c.n_rp, NTD, smem, stream>>>(p, c);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

// Worst-case number of workspace slots a tile needs for a given split.
int slots_needed(int tiles, int g_total, int gp, int n_rp, int CH) {
  int total = 0;
  for (int v = 0; v < g_total; v += gp) {
    const long Gq = (g_total - v) < gp ? (g_total - v) : gp;
    const long Cq = (Gq + CH - 1) / CH;
    const long Uq = (long)tiles * Cq;
    long Wq = (long)n_rp * NW;
    if (Wq > Uq) Wq = Uq;
    const long per_warp = Uq / Wq;           // >= 1
    total += (int)((Cq + per_warp - 1) / per_warp) + 1;
  }
  return total;
}

}  // namespace

int decode_supported(const Params& p) {
  if (p.M < 1 || p.M > 16) return 0;
  long tiles = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    if (job_tiles(p.job[j]) < 1) return 0;
    tiles += job_tiles(p.job[j]);
  }
  return tiles <= kCounterInts;
}

size_t decode_workspace_bytes(int M, int K, int N_total) {
  // arrival counters + fp32 partial sums: up to 4 slots of [M][16] per 16-row tile and k-part
  (void)K;
  size_t tiles = (size_t)(N_total + 15) / 16 + 8 * kMaxJobs;
  return (size_t)kCounterInts * 4 + tiles * (4 * kMaxKParts) * (size_t)M * 16 * 4;
}

int launch_decode(const Params& p, const LaunchCfg& cfg) {
  DecodeCfg c;
  memset(&c, 0, sizeof(c));
  build_spans(p.imap, &c);
  const int MT = p.M <= 8 ? 1 : 2;
  const int CH = MT == 1 ? 4 : 2;
  c.mp = MT == 1 ? p.M : 16;
  // 128-bit staging: one leading family, everything 8-element aligned
  c.x_vec = p.imap.n_fam == 1 && p.imap.fam[0].count == 1 && (p.imap.fam[0].start % 8) == 0 &&
            (p.imap.fam[0].keep % 8) == 0 && (p.ldx % 8) == 0 && ((((uintptr_t)p.x) & 15) == 0);
  int tiles = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    c.tile_begin[j] = tiles;
    tiles += job_tiles(p.job[j]);
  }
  for (int j = p.n_jobs; j <= kMaxJobs; ++j) c.tile_begin[j] = tiles;
  c.tiles_total = tiles;
  if (tiles > kCounterInts) return UNIQL_ERR_SHAPE;

  // ---- k-parts: as few as let the staged activations fit in shared memory (gp a multiple of CH)
  int n_kp = env_int("UNIQL_DECODE_KP", 0);
  if (n_kp < 1) {
    n_kp = 1;
    while (n_kp < kMaxKParts) {
      int gp = ((c.g_total + n_kp - 1) / n_kp + CH - 1) / CH * CH;
      if (smem_bytes(c.mp, gp, MT) <= kSmemBudget) break;
      ++n_kp;
    }
  }
  if (n_kp > kMaxKParts) n_kp = kMaxKParts;
  c.gp = ((c.g_total + n_kp - 1) / n_kp + CH - 1) / CH * CH;
  c.n_kp = (c.g_total + c.gp - 1) / c.gp;
  if (smem_bytes(c.mp, c.gp, MT) > 220 * 1024) return UNIQL_ERR_UNSUPPORTED;
  int n_rp = env_int("UNIQL_DECODE_RP", 0);
  if (n_rp < 1) n_rp = sm_count() / c.n_kp;
  if (n_rp < 1) n_rp = 1;
  c.n_rp = n_rp;
  c.max_slots = slots_needed(tiles, c.g_total, c.gp, c.n_rp, CH);
  {
    const size_t need = (size_t)kCounterInts * 4 + (size_t)tiles * c.max_slots * p.M * 16 * 4;
    if (!cfg.workspace || cfg.ws_bytes < need) return UNIQL_ERR_WORKSPACE;
  }
  // vector loads of scales / zero-points: every chunk starts CH-aligned in stored groups and is contiguous
  {
    const int G = p.K / kGroup;
    bool ok = c.n_spans == 1 && (c.vg_first[0] % CH) == 0 && (G % CH) == 0;
    for (int j = 0; j < p.n_jobs && ok; ++j)
      ok = ((((uintptr_t)p.job[j].scales) | ((uintptr_t)p.job[j].zeros)) & 15) == 0;
    c.sz_vec = ok;
  }
  c.counters = reinterpret_cast<int*>(cfg.workspace);
  c.partials = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(cfg.workspace) + (size_t)kCounterInts * 4);
  if (p.dt == UNIQL_F16)
    return MT == 1 ? launch_t<__half, 1, 4>(p, c, cfg.stream) : launch_t<__half, 2, 2>(p, c, cfg.stream);
  return MT == 1 ? launch_t<__nv_bfloat16, 1, 4>(p, c, cfg.stream) : launch_t<__nv_bfloat16, 2, 2>(p, c, cfg.stream);
}

}  // namespace uniql
