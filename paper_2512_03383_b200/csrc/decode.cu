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
// activation.  A thread block is wr x wk warps (row tiles x k-chunks); k-chunks of a block are
// reduced through shared memory, k-slices of different blocks through a workspace where the last
// block to arrive adds the partials in slice order (deterministic, no spinning).
// The rotary epilogue (Section 3.2, fused RoPE) needs both members of a rotation pair: in rope mode
// a 16-row tile is 8 pairs, first-half members in rows 0..7 and their partners in rows 8..15, which
// is exactly the (r, r+8) row pair a lane owns in the MMA accumulator layout.
#include <stdlib.h>

#include "common.cuh"

namespace uniql {
namespace {

constexpr int NTD = 128;          // threads per block (4 warps)
constexpr int kMaxSpans = kMaxFam;
constexpr int kCounterInts = 1 << 16;   // arrival counters at the head of the workspace

struct DecodeCfg {
  int wr, wk, gs;        // warps over rows, warps over k, groups per warp
  int n_slices;          // blocks along k
  int rb_total;
  int rb_begin[kMaxJobs + 1];
  int g_total;           // visited 128-channel groups
  int n_spans;
  int vg_begin[kMaxSpans + 1];  // visit index at which span s starts
  int vg_first[kMaxSpans];      // its first stored group
  int x_vec;             // activations can be staged with 128-bit loads
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

template <typename T> struct Cvt;
// fp16: a nibble in bits [3:0] of a 16-bit half ORed onto 0x6400 reads 1024+q, one in bits [7:4]
// ORed onto 0x5400 reads 64+q; subtracting 1032 / 72 leaves q-8 exactly.
template <> struct Cvt<__half> {
  static __device__ inline void word(uint32_t w, uint32_t (&a)[4]) {
    const __half2 k_lo = __halves2half2(__ushort_as_half(0x6408), __ushort_as_half(0x6408));  // 1032
    const __half2 k_hi = __halves2half2(__ushort_as_half(0x5480), __ushort_as_half(0x5480));  // 72
    uint32_t t0 = (w & 0x000f000fu) | 0x64006400u;
    uint32_t t1 = (w & 0x00f000f0u) | 0x54005400u;
    uint32_t w8 = w >> 8;
    uint32_t t2 = (w8 & 0x000f000fu) | 0x64006400u;
    uint32_t t3 = (w8 & 0x00f000f0u) | 0x54005400u;
    __half2 h0 = __hsub2(*reinterpret_cast<__half2*>(&t0), k_lo);
    __half2 h1 = __hsub2(*reinterpret_cast<__half2*>(&t1), k_hi);
    __half2 h2 = __hsub2(*reinterpret_cast<__half2*>(&t2), k_lo);
    __half2 h3 = __hsub2(*reinterpret_cast<__half2*>(&t3), k_hi);
    a[0] = *reinterpret_cast<uint32_t*>(&h0); a[1] = *reinterpret_cast<uint32_t*>(&h1);
    a[2] = *reinterpret_cast<uint32_t*>(&h2); a[3] = *reinterpret_cast<uint32_t*>(&h3);
  }
  static __device__ inline void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                    uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
};
// bf16 has 7 mantissa bits: only a nibble in bits [3:0] can be ORed onto 0x4300 (128+q).
template <> struct Cvt<__nv_bfloat16> {
  static __device__ inline void word(uint32_t w, uint32_t (&a)[4]) {
    const __nv_bfloat162 k136 = __halves2bfloat162(__ushort_as_bfloat16(0x4308), __ushort_as_bfloat16(0x4308));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t t = ((w >> (4 * i)) & 0x000f000fu) | 0x43004300u;
      __nv_bfloat162 h = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&t), k136);
      a[i] = *reinterpret_cast<uint32_t*>(&h);
    }
  }
  static __device__ inline void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                    uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
};

// 16-byte unit of the staged activations: local group lv, activation row m, word j, lane chunk c.
// The XOR keeps the eight lanes of a 128-bit shared load phase on distinct banks.
__device__ inline int x_unit(int lv, int mp, int m, int j, int c) {
  return (lv * mp + m) * 16 + (((j ^ (m & 1)) << 2) | c);
}

struct GroupLoad {
  uint4 w0, w1;        // 32 codes of rows r and r+8
  float s0, z0, s1, z1;
};

template <typename T, int MT>
__global__ void __launch_bounds__(NTD) decode_kernel(const __grid_constant__ Params p,
                                                     const __grid_constant__ DecodeCfg c) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = lane >> 2, cq = lane & 3;
  const int mp = c.mp;
  const int WG = c.wk * c.gs;
  uint4* xs = reinterpret_cast<uint4*>(smem);
  float* xg = reinterpret_cast<float*>(smem + (size_t)WG * mp * 256);   // [WG][mp]

  const int rb = blockIdx.x;
  int jn = 0;
  while (jn + 1 < p.n_jobs && rb >= c.rb_begin[jn + 1]) ++jn;
  const JobDev& jb = p.job[jn];
  const int wr_i = warp % c.wr, wk_i = warp / c.wr;
  const int tile = (rb - c.rb_begin[jn]) * c.wr + wr_i;

  // ---- the two weight rows of this lane: stored row (clamped for loads) and output column
  int sr0, sr1, oc0, oc1, rope_p = 0, rope_kvh = 0;
  if (jb.rope.enabled) {
    const int half = jb.rope.head_keep >> 1;
    const int P = tile * 8 + r;
    const bool ok = P < jb.rope.n_heads * half;
    const int Pc = ok ? P : 0;
    const int h = Pc / half, cc = Pc - h * half;
    sr0 = h * jb.rope.head_dim + cc;
    sr1 = sr0 + (jb.rope.head_dim >> 1);
    oc0 = ok ? h * jb.rope.head_keep + cc : -1;
    oc1 = ok ? oc0 + half : -1;
    rope_p = cc;
    rope_kvh = h / jb.rope.rep;
  } else {
    const int j0 = tile * 16 + r, j1 = j0 + 8;
    oc0 = j0 < jb.k_out ? j0 : -1;
    oc1 = j1 < jb.k_out ? j1 : -1;
    sr0 = map_compact_to_stored(jb.omap, oc0 >= 0 ? j0 : 0);
    sr1 = map_compact_to_stored(jb.omap, oc1 >= 0 ? j1 : 0);
  }
  const int G = p.K / kGroup;
  const uint8_t* wrow0 = jb.w + (size_t)sr0 * (p.K / 2) + cq * 16;
  const uint8_t* wrow1 = jb.w + (size_t)sr1 * (p.K / 2) + cq * 16;
  const __half* srow0 = jb.scales + (size_t)sr0 * G;
  const __half* zrow0 = jb.zeros + (size_t)sr0 * G;
  const __half* srow1 = jb.scales + (size_t)sr1 * G;
  const __half* zrow1 = jb.zeros + (size_t)sr1 * G;

  const int cta_v0 = blockIdx.y * WG;           // first visit index of this block
  const int lv0 = wk_i * c.gs;                  // first local group of this warp

  auto load_group = [&](int lv) -> GroupLoad {
    GroupLoad g;
    const int v = cta_v0 + lv;
    if (lv < lv0 + c.gs && v < c.g_total) {
      const int sg = visit_to_group(c, v);
      g.w0 = ldg_stream(wrow0 + (size_t)sg * 64);
      g.w1 = ldg_stream(wrow1 + (size_t)sg * 64);
      g.s0 = __half2float(__ldg(srow0 + sg)); g.z0 = __half2float(__ldg(zrow0 + sg)) - 8.f;
      g.s1 = __half2float(__ldg(srow1 + sg)); g.z1 = __half2float(__ldg(zrow1 + sg)) - 8.f;
    } else {
      g.w0 = make_uint4(0, 0, 0, 0); g.w1 = g.w0;
      g.s0 = g.z0 = g.s1 = g.z1 = 0.f;
    }
    return g;
  };

  // first weight loads go out before the activations are staged (they do not depend on them)
  GroupLoad cur0 = load_group(lv0), cur1 = load_group(lv0 + 1);

  // ---- stage activations: permuted into nibble order, zero where the channel is pruned
  {
    const T* x = reinterpret_cast<const T*>(p.x);
    if (c.x_vec) {
      const int start = p.imap.fam[0].start, keep = p.imap.fam[0].keep;
      const int n_units = WG * mp * 16;
      for (int u = tid; u < ((n_units + 31) & ~31); u += NTD) {   // whole warps stay in the shuffles
        const bool in_range = u < n_units;
        const int u16 = u & 15, pair = in_range ? u >> 4 : 0;
        const int lv = pair / mp, m = pair - lv * mp;
        const int ccq = u16 >> 2, j = u16 & 3;
        const int v = cta_v0 + lv;
        uint4 in = make_uint4(0, 0, 0, 0);
        if (in_range && v < c.g_total && m < p.M) {
          const int t0 = visit_to_group(c, v) * kGroup + 8 * u16 - start;
          if (t0 >= 0 && t0 < keep) in = *reinterpret_cast<const uint4*>(x + (size_t)m * p.ldx + t0);
        }
        uint4 o;
        o.x = __byte_perm(in.x, in.z, 0x5410); o.y = __byte_perm(in.x, in.z, 0x7632);
        o.z = __byte_perm(in.y, in.w, 0x5410); o.w = __byte_perm(in.y, in.w, 0x7632);
        if (in_range) xs[x_unit(lv, mp, m, j, ccq)] = o;
        const typename DT<T>::T2* h2 = reinterpret_cast<const typename DT<T>::T2*>(&in);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 f = DT<T>::to_f2(h2[i]); sum += f.x + f.y; }
#pragma unroll
        for (int o2 = 8; o2 >= 1; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
        if (in_range && u16 == 0) xg[pair] = sum;
      }
    } else {
      T* xh = reinterpret_cast<T*>(smem);
      const int n_pairs = WG * mp;
      for (int pair = warp; pair < n_pairs; pair += NTD / 32) {
        const int lv = pair / mp, m = pair - lv * mp;
        const int v = cta_v0 + lv;
        const bool live = v < c.g_total && m < p.M;
        const int kbase = live ? visit_to_group(c, v) * kGroup : 0;
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
          xh[x_unit(lv, mp, m, j, ccq) * 8 + 2 * (e & 3) + (e >> 2)] = val;
          sum += DT<T>::to_f(val);
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
        if (lane == 0) xg[pair] = sum;
      }
    }
  }
  __syncthreads();

  // ---- main loop over this warp's groups, two groups of loads in flight ahead of the math
  float out[MT][4];
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) out[t][i] = 0.f;

  auto process = [&](const GroupLoad& g, int lv) {
    float acc[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;
    const uint32_t w0[4] = {g.w0.x, g.w0.y, g.w0.z, g.w0.w};
    const uint32_t w1[4] = {g.w1.x, g.w1.y, g.w1.z, g.w1.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t a[4], b[4];
      Cvt<T>::word(w0[j], a);
      Cvt<T>::word(w1[j], b);
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        const int m = r + 8 * t;
        uint4 xb = make_uint4(0, 0, 0, 0);
        if (m < mp) xb = xs[x_unit(lv, mp, m, j, cq)];
        Cvt<T>::mma(acc[t], a[0], b[0], a[1], b[1], xb.x, xb.y);
        Cvt<T>::mma(acc[t], a[2], b[2], a[3], b[3], xb.z, xb.w);
      }
    }
#pragma unroll
    for (int t = 0; t < MT; ++t) {
      const int m0 = 2 * cq + 8 * t;
      const float X0 = m0 < mp ? xg[lv * mp + m0] : 0.f;
      const float X1 = m0 + 1 < mp ? xg[lv * mp + m0 + 1] : 0.f;
      out[t][0] = fmaf(g.s0, fmaf(-g.z0, X0, acc[t][0]), out[t][0]);
      out[t][1] = fmaf(g.s0, fmaf(-g.z0, X1, acc[t][1]), out[t][1]);
      out[t][2] = fmaf(g.s1, fmaf(-g.z1, X0, acc[t][2]), out[t][2]);
      out[t][3] = fmaf(g.s1, fmaf(-g.z1, X1, acc[t][3]), out[t][3]);
    }
  };

  for (int i = 0; i < c.gs; i += 2) {
    GroupLoad nxt0 = load_group(lv0 + i + 2), nxt1 = load_group(lv0 + i + 3);
    process(cur0, lv0 + i);
    if (i + 1 < c.gs) process(cur1, lv0 + i + 1);
    cur0 = nxt0; cur1 = nxt1;
  }

  // ---- reduce the k-chunks of this block through shared memory
  if (c.wk > 1) {
    __syncthreads();
    float* red = reinterpret_cast<float*>(smem);
    if (wk_i > 0) {
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) red[(((wk_i - 1) * c.wr + wr_i) * 32 + lane) * (MT * 4) + t * 4 + i] = out[t][i];
    }
    __syncthreads();
    if (wk_i == 0) {
      for (int k = 1; k < c.wk; ++k)
#pragma unroll
        for (int t = 0; t < MT; ++t)
#pragma unroll
          for (int i = 0; i < 4; ++i) out[t][i] += red[(((k - 1) * c.wr + wr_i) * 32 + lane) * (MT * 4) + t * 4 + i];
    }
  }
  const bool active = wk_i == 0;

  // ---- reduce the k-slices of different blocks: the last block to arrive sums in slice order
  if (c.n_slices > 1) {
    __shared__ int s_last;
    float4* part = reinterpret_cast<float4*>(c.partials);
    const size_t slot = ((size_t)rb * c.wr + wr_i) * 32 + lane;
    const size_t slice_stride = (size_t)c.rb_total * c.wr * 32;
    if (active) {
#pragma unroll
      for (int t = 0; t < MT; ++t)
        __stcg(&part[((size_t)blockIdx.y * slice_stride + slot) * MT + t],
               make_float4(out[t][0], out[t][1], out[t][2], out[t][3]));
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int ticket = atomicAdd(&c.counters[rb], 1);
      s_last = ticket == c.n_slices - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (active) {
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) out[t][i] = 0.f;
      for (int s = 0; s < c.n_slices; ++s)
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          const float4 v = __ldcg(&part[((size_t)s * slice_stride + slot) * MT + t]);
          out[t][0] += v.x; out[t][1] += v.y; out[t][2] += v.z; out[t][3] += v.w;
        }
    }
    if (tid == 0) c.counters[rb] = 0;     // ready for the next call
  }
  if (!active) return;

  // ---- epilogue: bias, rotary embedding on the retained pair, one rounding, store
  const T* bias = reinterpret_cast<const T*>(jb.bias);
  const float b0 = (bias && oc0 >= 0) ? DT<T>::to_f(bias[sr0]) : 0.f;
  const float b1 = (bias && oc1 >= 0) ? DT<T>::to_f(bias[sr1]) : 0.f;
  T* y = reinterpret_cast<T*>(jb.y);
  double invf = 0.0;
  if (jb.rope.enabled) {
    int pidx = p.idx[rope_kvh * (jb.rope.head_keep >> 1) + rope_p];
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
      if (oc0 >= 0) y[(size_t)m * jb.ldy + oc0] = DT<T>::from_f(lo);
      if (oc1 >= 0) y[(size_t)m * jb.ldy + oc1] = DT<T>::from_f(hi);
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

int row_blocks(const Params& p, int wr, int* begin) {
  int tot = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    begin[j] = tot;
    tot += (job_tiles(p.job[j]) + wr - 1) / wr;
  }
  for (int j = p.n_jobs; j <= kMaxJobs; ++j) begin[j] = tot;
  return tot;
}

}  // namespace

int decode_supported(const Params& p) {
  if (p.M < 1 || p.M > 16) return 0;
  for (int j = 0; j < p.n_jobs; ++j)
    if (job_tiles(p.job[j]) < 1) return 0;
  return 1;
}

size_t decode_workspace_bytes(int M, int K, int N_total) {
  // counters + up to 16 k-slices of fp32 partials for every 16-row tile (padded per job)
  (void)K;
  size_t mt = M <= 8 ? 1 : 2;
  size_t tiles = (size_t)(N_total + 15) / 16 + 4 * kMaxJobs;
  return (size_t)kCounterInts * 4 + 16 * tiles * 32 * mt * 16;
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

  const size_t ws_part = cfg.ws_bytes > (size_t)kCounterInts * 4 ? cfg.ws_bytes - (size_t)kCounterInts * 4 : 0;
  const int force_wk = env_int("UNIQL_DECODE_WK", 0), force_gs = env_int("UNIQL_DECODE_GS", 0);
  double best = -1.0;
  int bwk = 0, bgs = 0;
  const int wks[3] = {4, 2, 1};
  const int gss[5] = {8, 4, 2, 16, 1};
  for (int a = 0; a < 3; ++a)
    for (int b = 0; b < 5; ++b) {
      int wk = wks[a], gs = gss[b], wr = 4 / wk;
      if (force_wk && wk != force_wk) continue;
      if (force_gs && gs != force_gs) continue;
      int WG = wk * gs;
      size_t smem = (size_t)WG * c.mp * 256 + (size_t)WG * c.mp * 4;
      if (smem > 64 * 1024) continue;
      int slices = (c.g_total + WG - 1) / WG;
      int begin[kMaxJobs + 1];
      int rbt = row_blocks(p, wr, begin);
      if (rbt > kCounterInts) continue;
      if (slices > 1) {
        size_t need = (size_t)slices * rbt * wr * 32 * MT * 16;
        if (need > ws_part) continue;
      }
      if (slices > 65535) continue;
      double useful = (double)c.g_total / ((double)slices * WG);
      double ctas = (double)rbt * slices;
      const double slots = 148.0 * 4.0;
      double waves = ceil(ctas / slots);
      double wave_eff = ctas / (waves * slots);
      double score = useful * wave_eff;
      if (slices > 1) score *= 1.0 - 0.01 * p.M;     // partial-sum traffic grows with M
      score *= 1.0 + 0.01 * (gs >= 4 ? 1.0 : 0.0);    // prefer enough loads in flight per warp
      if (score > best) { best = score; bwk = wk; bgs = gs; }
    }
  if (best < 0) return UNIQL_ERR_WORKSPACE;
  c.wk = bwk; c.gs = bgs; c.wr = 4 / bwk;
  const int WG = c.wk * c.gs;
  c.n_slices = (c.g_total + WG - 1) / WG;
  c.rb_total = row_blocks(p, c.wr, c.rb_begin);
  c.counters = reinterpret_cast<int*>(cfg.workspace);
  c.partials = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(cfg.workspace) + (size_t)kCounterInts * 4);
  if (c.n_slices > 1 && !cfg.workspace) return UNIQL_ERR_WORKSPACE;

  size_t smem = (size_t)WG * c.mp * 256 + (size_t)WG * c.mp * 4;
  size_t red = (size_t)4 * 32 * MT * 16;
  if (smem < red) smem = red;
  dim3 grid(c.rb_total, c.n_slices);
  auto launch = [&](auto kern) -> int {
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return UNIQL_ERR_CUDA;
    kern<<<grid, NTD, smem, cfg.stream>>>(p, c);
    return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
  };
  if (p.dt == UNIQL_F16)
    return MT == 1 ? launch(decode_kernel<__half, 1>) : launch(decode_kernel<__half, 2>);
  return MT == 1 ? launch(decode_kernel<__nv_bfloat16, 1>) : launch(decode_kernel<__nv_bfloat16, 2>);
}

}  // namespace uniql
