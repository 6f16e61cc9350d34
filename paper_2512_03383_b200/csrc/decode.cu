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
// activation.  A block of four warps owns one k-slice of GS groups (its activations staged once)
// and walks over 4*tpw row tiles; a warp issues all 2*GS loads of a tile before it touches them,
// and the other resident warps hide the latency.  k-slices of different blocks meet in a workspace
// where the last block to arrive adds the partials in slice order (deterministic, no spinning).
// The rotary epilogue (Section 3.2, fused RoPE) needs both members of a rotation pair: in rope mode
// a 16-row tile is 8 pairs, first-half members in rows 0..7 and their partners in rows 8..15, which
// is exactly the (r, r+8) row pair a lane owns in the MMA accumulator layout.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace uniql {
namespace {

constexpr int NTD = 128;          // threads per block (4 warps)
constexpr int kMaxSpans = kMaxFam;
constexpr int kCounterInts = 1 << 16;   // arrival counters at the head of the workspace

struct DecodeCfg {
  int tpw;               // row tiles per warp
  int n_slices;          // blocks along k
  int rb_total;
  int rb_begin[kMaxJobs + 1];
  int tiles[kMaxJobs];
  int row_base[kMaxJobs];   // first row of each job in the partial-sum buffer
  int rows_total;
  int g_total;           // visited 128-channel groups
  int n_spans;
  int vg_begin[kMaxSpans + 1];  // visit index at which span s starts
  int vg_first[kMaxSpans];      // its first stored group
  int x_vec;             // activations can be staged with 128-bit loads
  int sz_vec;            // scales / zero-points of a slice can be fetched with one vector load
  int mp;                // activation rows staged in shared memory
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

// 16-byte unit of the staged activations: activation row m, local group lv, word j, lane chunk c.
// A row holds GS groups of 256 bytes plus 64 bytes of padding, so that the two rows met by the eight
// lanes of one 128-bit shared-load phase sit 64 bytes apart modulo 128 (distinct banks), and every
// (group, word) offset is a compile-time immediate.
template <int GS>
__device__ inline int x_unit(int lv, int m, int j, int c) {
  return m * (GS * 16 + 4) + lv * 16 + j * 4 + c;
}

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

template <typename T, int MT, int GS>
__global__ void __launch_bounds__(NTD) decode_kernel(const __grid_constant__ Params p,
                                                     const __grid_constant__ DecodeCfg c) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = lane >> 2, cq = lane & 3;
  const int mp = c.mp;
  // shared memory: staged activations, mp rows + one all-zero row of (GS*256+64) bytes each, then
  // the per-group activation sums [GS][8*MT] fp32
  constexpr int kRowBytes = GS * 256 + 64;
  uint4* xs = reinterpret_cast<uint4*>(smem);
  const int xg_off = (mp + 1) * kRowBytes;
  float* xg = reinterpret_cast<float*>(smem + xg_off);

  const int rb = blockIdx.x;
  int jn = 0;
  while (jn + 1 < p.n_jobs && rb >= c.rb_begin[jn + 1]) ++jn;
  const JobDev& jb = p.job[jn];
  const int v0 = blockIdx.y * GS;
  const int nvalid = min(GS, c.g_total - v0);
  const int sg0 = visit_to_group(c, v0);
  const bool contig = visit_to_group(c, v0 + nvalid - 1) == sg0 + nvalid - 1;   // block-uniform

  // ---- stage activations: permuted into nibble order, zero where the channel is pruned
  {
    const T* x = reinterpret_cast<const T*>(p.x);
    for (int i = tid; i < kRowBytes / 16; i += NTD) xs[mp * (kRowBytes / 16) + i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < GS * 8 * MT; i += NTD) xg[i] = 0.f;
    __syncthreads();
    if (c.x_vec) {
      const int start = p.imap.fam[0].start, keep = p.imap.fam[0].keep;
      const int n_units = GS * mp * 16;
      for (int u = tid; u < ((n_units + 31) & ~31); u += NTD) {   // whole warps stay in the shuffles
        const bool in_range = u < n_units;
        const int u16 = u & 15, pair = in_range ? u >> 4 : 0;
        const int m = pair / GS, lv = pair - m * GS;
        const int ccq = u16 >> 2, j = u16 & 3;
        uint4 in = make_uint4(0, 0, 0, 0);
        if (in_range && lv < nvalid && m < p.M) {
          const int t0 = (contig ? sg0 + lv : visit_to_group(c, v0 + lv)) * kGroup + 8 * u16 - start;
          if (t0 >= 0 && t0 < keep) in = *reinterpret_cast<const uint4*>(x + (size_t)m * p.ldx + t0);
        }
        uint4 o;
        o.x = __byte_perm(in.x, in.z, 0x5410); o.y = __byte_perm(in.x, in.z, 0x7632);
        o.z = __byte_perm(in.y, in.w, 0x5410); o.w = __byte_perm(in.y, in.w, 0x7632);
        if (in_range) xs[x_unit<GS>(lv, m, j, ccq)] = o;
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
      const int n_pairs = GS * mp;
      for (int pair = warp; pair < n_pairs; pair += NTD / 32) {
        const int m = pair / GS, lv = pair - m * GS;
        const bool live = lv < nvalid && m < p.M;
        const int kbase = live ? visit_to_group(c, v0 + lv) * kGroup : 0;
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
          xh[x_unit<GS>(lv, m, j, ccq) * 8 + 2 * (e & 3) + (e >> 2)] = val;
          sum += DT<T>::to_f(val);
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
        if (lane == 0) xg[lv * 8 * MT + m] = sum;
      }
    }
  }
  __syncthreads();

  // per-lane shared-memory address of the B fragments (lanes beyond the staged rows read the zero row)
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
  uint32_t xb_addr[MT];
#pragma unroll
  for (int t = 0; t < MT; ++t) {
    const int m = r + 8 * t;
    xb_addr[t] = smem_base + (uint32_t)((m < mp ? m : mp) * kRowBytes + cq * 16);
  }
  const uint32_t xg_addr = smem_base + (uint32_t)xg_off + (uint32_t)(2 * cq * 4);

  const int G = p.K / kGroup;
  const int first_tile = (rb - c.rb_begin[jn]) * (4 * c.tpw);
  const int n_tiles = c.tiles[jn];
  const size_t part_mstride = (size_t)c.rows_total;

  for (int it = 0; it < c.tpw; ++it) {
    const int tile = first_tile + it * 4 + warp;
    if (tile >= n_tiles) break;
    const LaneRows L = resolve_rows(jb, tile, r);
    const uint8_t* wrow0 = jb.w + (size_t)L.sr0 * (p.K / 2) + cq * 16;
    const uint8_t* wrow1 = jb.w + (size_t)L.sr1 * (p.K / 2) + cq * 16;

    // ---- all loads of this tile first
    uint4 w0[GS], w1[GS];
    if (contig) {
      const uint8_t* q0 = wrow0 + (size_t)sg0 * 64;
      const uint8_t* q1 = wrow1 + (size_t)sg0 * 64;
#pragma unroll
      for (int g = 0; g < GS; ++g) {
        if (g < nvalid) {
          w0[g] = ldg_stream(q0 + g * 64);
          w1[g] = ldg_stream(q1 + g * 64);
        } else {
          w0[g] = make_uint4(0, 0, 0, 0); w1[g] = w0[g];
        }
      }
    } else {
#pragma unroll
      for (int g = 0; g < GS; ++g) {
        if (g < nvalid) {
          const size_t off = (size_t)visit_to_group(c, v0 + g) * 64;
          w0[g] = ldg_stream(wrow0 + off);
          w1[g] = ldg_stream(wrow1 + off);
        } else {
          w0[g] = make_uint4(0, 0, 0, 0); w1[g] = w0[g];
        }
      }
    }
    uint32_t sc[4][(GS + 1) / 2];   // packed fp16 pairs: s(row r), z(row r), s(row r+8), z(row r+8)
    {
      const __half* base[4] = {jb.scales + (size_t)L.sr0 * G, jb.zeros + (size_t)L.sr0 * G,
                               jb.scales + (size_t)L.sr1 * G, jb.zeros + (size_t)L.sr1 * G};
      if (c.sz_vec) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if constexpr (GS == 8) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(base[q] + sg0));
            sc[q][0] = v.x; sc[q][1] = v.y; sc[q][2] = v.z; sc[q][3] = v.w;
          } else if constexpr (GS == 4) {
            const uint2 v = __ldg(reinterpret_cast<const uint2*>(base[q] + sg0));
            sc[q][0] = v.x; sc[q][1] = v.y;
          } else {
            sc[q][0] = __ldg(reinterpret_cast<const uint32_t*>(base[q] + sg0));
          }
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int g = 0; g < GS; g += 2) {
            const int ga = visit_to_group(c, v0 + (g < nvalid ? g : 0));
            const int gb = visit_to_group(c, v0 + (g + 1 < nvalid ? g + 1 : 0));
            const uint32_t lo = __half_as_ushort(__ldg(base[q] + ga));
            const uint32_t hi = __half_as_ushort(__ldg(base[q] + gb));
            sc[q][g >> 1] = lo | (hi << 16);
          }
      }
    }

    float out[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) out[t][i] = 0.f;

#pragma unroll
    for (int g = 0; g < GS; ++g) {
      if (g < nvalid) {
        // two accumulators per batch tile keep two independent MMA chains in flight
        float acc[MT][2][4];
        const uint32_t wa[4] = {w0[g].x, w0[g].y, w0[g].z, w0[g].w};
        const uint32_t wb[4] = {w1[g].x, w1[g].y, w1[g].z, w1[g].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t a[4], b[4];
          Cvt<T>::word(wa[j], a);
          Cvt<T>::word(wb[j], b);
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            const uint4 xb = lds128(xb_addr[t] + (uint32_t)(g * 256 + j * 64));
            if (j == 0) {
              Cvt<T>::mma0(acc[t][0], a[0], b[0], a[1], b[1], xb.x, xb.y);
              Cvt<T>::mma0(acc[t][1], a[2], b[2], a[3], b[3], xb.z, xb.w);
            } else {
              Cvt<T>::mma(acc[t][0], a[0], b[0], a[1], b[1], xb.x, xb.y);
              Cvt<T>::mma(acc[t][1], a[2], b[2], a[3], b[3], xb.z, xb.w);
            }
          }
        }
        auto pick = [&](int q) -> float {
          const __half2 h = *reinterpret_cast<const __half2*>(&sc[q][g >> 1]);
          return (g & 1) ? __high2float(h) : __low2float(h);
        };
        const float s0 = pick(0), nz0 = 8.f - pick(1);
        const float s1 = pick(2), nz1 = 8.f - pick(3);
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          const float2 X = lds64f(xg_addr + (uint32_t)((g * 8 * MT + 8 * t) * 4));
          out[t][0] = fmaf(s0, fmaf(nz0, X.x, acc[t][0][0] + acc[t][1][0]), out[t][0]);
          out[t][1] = fmaf(s0, fmaf(nz0, X.y, acc[t][0][1] + acc[t][1][1]), out[t][1]);
          out[t][2] = fmaf(s1, fmaf(nz1, X.x, acc[t][0][2] + acc[t][1][2]), out[t][2]);
          out[t][3] = fmaf(s1, fmaf(nz1, X.y, acc[t][0][3] + acc[t][1][3]), out[t][3]);
        }
      }
    }

    if (c.n_slices == 1) {
      epilogue<T, MT>(p, jb, L, cq, out);
    } else {
      // compact partial sums: [slice][m][row]
      float* part = c.partials + (size_t)blockIdx.y * p.M * part_mstride + c.row_base[jn];
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int m = 2 * cq + e + 8 * t;
          if (m >= p.M) continue;
          if (L.oc0 >= 0) __stcg(part + (size_t)m * part_mstride + L.oc0, out[t][e]);
          if (L.oc1 >= 0) __stcg(part + (size_t)m * part_mstride + L.oc1, out[t][2 + e]);
        }
    }
  }
  if (c.n_slices == 1) return;

  // ---- the last block to arrive for this row block sums the slices in order and finishes
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&c.counters[rb], 1);
    s_last = ticket == c.n_slices - 1;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int it = 0; it < c.tpw; ++it) {
    const int tile = first_tile + it * 4 + warp;
    if (tile >= n_tiles) break;
    const LaneRows L = resolve_rows(jb, tile, r);
    float out[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) out[t][i] = 0.f;
    for (int s = 0; s < c.n_slices; ++s) {
      const float* part = c.partials + (size_t)s * p.M * part_mstride + c.row_base[jn];
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int m = 2 * cq + e + 8 * t;
          if (m >= p.M) continue;
          if (L.oc0 >= 0) out[t][e] += __ldcg(part + (size_t)m * part_mstride + L.oc0);
          if (L.oc1 >= 0) out[t][2 + e] += __ldcg(part + (size_t)m * part_mstride + L.oc1);
        }
    }
    epilogue<T, MT>(p, jb, L, cq, out);
  }
  if (tid == 0) c.counters[rb] = 0;     // ready for the next call
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

template <typename T, int MT, int GS>
int launch_t(const Params& p, const DecodeCfg& c, cudaStream_t stream) {
  size_t smem = (size_t)(c.mp + 1) * (GS * 256 + 64) + (size_t)GS * 8 * MT * 4;
  auto kern = decode_kernel<T, MT, GS>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return UNIQL_ERR_CUDA;
  dim3 grid(c.rb_total, c.n_slices);
  kern<<<grid, NTD, smem, stream>>>(p, c);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

template <typename T>
int launch_dt(const Params& p, const DecodeCfg& c, int MT, int GS, cudaStream_t stream) {
  if (MT == 1) {
    if (GS == 8) return launch_t<T, 1, 8>(p, c, stream);
    if (GS == 4) return launch_t<T, 1, 4>(p, c, stream);
    return launch_t<T, 1, 2>(p, c, stream);
  }
  if (GS == 8) return launch_t<T, 2, 8>(p, c, stream);
  if (GS == 4) return launch_t<T, 2, 4>(p, c, stream);
  return launch_t<T, 2, 2>(p, c, stream);
}

}  // namespace

int decode_supported(const Params& p) {
  if (p.M < 1 || p.M > 16) return 0;
  for (int j = 0; j < p.n_jobs; ++j)
    if (job_tiles(p.job[j]) < 1) return 0;
  return 1;
}

size_t decode_workspace_bytes(int M, int K, int N_total) {
  // counters + fp32 partial sums [slices][M][rows] for the finest slicing (2 groups per slice)
  size_t slices = (size_t)(K / kGroup + 1) / 2 + 1;
  return (size_t)kCounterInts * 4 + slices * (size_t)M * (size_t)N_total * 4;
}

int launch_decode(const Params& p, const LaunchCfg& cfg) {
  DecodeCfg c;
  memset(&c, 0, sizeof(c));
  build_spans(p.imap, &c);
  const int MT = p.M <= 8 ? 1 : 2;
  c.mp = MT == 1 ? p.M : 16;
  // 128-bit staging: one leading family, everything 8-element aligned
  c.x_vec = p.imap.n_fam == 1 && p.imap.fam[0].count == 1 && (p.imap.fam[0].start % 8) == 0 &&
            (p.imap.fam[0].keep % 8) == 0 && (p.ldx % 8) == 0 && ((((uintptr_t)p.x) & 15) == 0);
  int rows = 0, tiles_total = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    c.tiles[j] = job_tiles(p.job[j]);
    c.row_base[j] = rows;
    rows += p.job[j].k_out;
    tiles_total += c.tiles[j];
  }
  c.rows_total = rows;

  const size_t ws_part = cfg.ws_bytes > (size_t)kCounterInts * 4 ? cfg.ws_bytes - (size_t)kCounterInts * 4 : 0;
  // ---- block shape: GS groups per k-slice, tpw row tiles per warp
  const int force_gs = env_int("UNIQL_DECODE_GS", 0), force_tpw = env_int("UNIQL_DECODE_TPW", 0);
  int GS = MT == 1 ? 8 : 4;
  if (c.g_total < GS) GS = c.g_total >= 4 ? 4 : 2;
  if (force_gs == 8 || force_gs == 4 || force_gs == 2) GS = force_gs;
  int slices = (c.g_total + GS - 1) / GS;
  while (slices > 1 && (size_t)slices * p.M * rows * 4 > ws_part && GS < 8) {   // coarser slices need less workspace
    GS *= 2;
    slices = (c.g_total + GS - 1) / GS;
  }
  if (slices > 1 && (!cfg.workspace || (size_t)slices * p.M * rows * 4 > ws_part)) return UNIQL_ERR_WORKSPACE;
  if (slices > 65535) return UNIQL_ERR_SHAPE;
  // enough blocks to fill the machine a few times over, otherwise as many tiles per warp as possible
  int tpw = 1;
  {
    const long target = 148L * 4 * 4;
    while (tpw < 8 && (long)((tiles_total + 4 * (tpw * 2) - 1) / (4 * (tpw * 2))) * slices >= target) tpw *= 2;
  }
  if (force_tpw >= 1 && force_tpw <= 64) tpw = force_tpw;
  c.tpw = tpw;
  c.n_slices = slices;
  int rbt = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    c.rb_begin[j] = rbt;
    rbt += (c.tiles[j] + 4 * tpw - 1) / (4 * tpw);
  }
  for (int j = p.n_jobs; j <= kMaxJobs; ++j) c.rb_begin[j] = rbt;
  c.rb_total = rbt;
  if (rbt > kCounterInts) return UNIQL_ERR_SHAPE;
  // vector loads of scales / zero-points: slice starts GS-aligned, contiguous, rows GS-aligned
  {
    const int G = p.K / kGroup;
    bool ok = c.n_spans == 1 && (c.vg_first[0] % GS) == 0 && (G % GS) == 0;
    for (int j = 0; j < p.n_jobs && ok; ++j)
      ok = ((((uintptr_t)p.job[j].scales) | ((uintptr_t)p.job[j].zeros)) & 15) == 0;
    c.sz_vec = ok;
  }
  c.counters = reinterpret_cast<int*>(cfg.workspace);
  c.partials = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(cfg.workspace) + (size_t)kCounterInts * 4);
  if (p.dt == UNIQL_F16) return launch_dt<__half>(p, c, MT, GS, cfg.stream);
  return launch_dt<__nv_bfloat16>(p, c, MT, GS, cfg.stream);
}

}  // namespace uniql
