// Streaming decode kernel for batches of one to four rows (fp16), sm_100a.
//
// At these batch sizes every retained weight is read once and used for at most four products: the launch is a
// stream of 4-bit codes from HBM, and what matters is that the stream is dense from the first microsecond to the
// last and that every SM carries the same share of it.
//
// Work.  A tile is 16 MMA rows, a step is GCH quantisation groups (512 input channels) of a tile: 4 KB of codes and
// their scales / zero-points.  The steps of all tiles form one sequence (tile after tile); it is cut into equal
// contiguous ranges, one per WARP of a persistent grid (one block of eight warps per SM), so every warp streams the
// same number of bytes whatever the shape.  A warp is its own pipeline: it copies its steps from global memory into
// a private shared-memory ring with asynchronous 16-byte copies, four steps ahead (sixteen lanes fetch 256
// contiguous bytes of a weight row; no registers held, no block-wide barrier, no other warp involved), and consumes
// them in order.  A tile whose steps fall into several warps' ranges is finished by the last of them to arrive:
// each parks its fp32 partial sums in the workspace, and the last one adds them in range order (deterministic).
//
// Activations.  The rings are filled before the dependency wait (weights are never produced by the preceding
// kernel); after it every block quantises the activations once into its shared memory: 16-bit fixed point per
// (batch row, 128-channel group), split into a high and a low signed byte, in the order the nibbles leave a
// weight word.  Activations are fetched in units of 4 channels, so kept blocks of 108 or 84 channels and blocks of
// 1740 leading channels need no re-laying.
//
// On-device pruning (Section 3.4) is index arithmetic: a tile only addresses kept rows, a step only visited input
// groups, and pruned input channels inside a visited group meet zero activations.
//
// Arithmetic (as in the persistent decode kernel): the codes go to the int8 tensor-core MMA as they lie in memory.
// Per 32-bit weight word three ALU operations give the low and the high nibbles as bytes, the A fragments of one
// m16n8k32 MMA for two weight rows; B holds the activation bytes (columns 2m and 2m+1 of the MMA are the high and
// the low byte of batch row m).  256 * d_hi + d_lo = sum q * x_i exactly; scale, zero-point and 2^-e are applied
// once per (row, group) in fp32:  y += s * 2^-e * (sum q x_i - z * sum x_i).
//
// MMA row g of a tile and row g + 8 are chosen so that an output needs both of them only inside one lane:
//   plain   rows r0 + g and r0 + 8 + g of a kept block;
//   rope    the two members of rotation pair c0 + g of one head (Section 3.2, fused RoPE on the retained pairs);
//   swiglu  row c0 + g of the gate matrix and of the up matrix (Section 3.2, MLP paragraph).
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "quant.cuh"

namespace uniql {
namespace {

constexpr int GW = 8;                    // warps per block, one block per SM
constexpr int GTH = GW * 32;
constexpr int GCH = 4;                   // groups per step
constexpr int kSlotW = 16 * GCH * 64;    // codes of a step: 16 MMA rows x 256 bytes
constexpr int kSlotBytes = kSlotW + 256; // ... + GCH scales and GCH zero-points of the 16 rows
constexpr int kGvMaxDepth = 5;           // ring slots per warp (steps in flight: depth - 1)
constexpr int kGvSmemMax = 225 * 1024;
constexpr int kGvMaxFam = 8;
constexpr int kGvCounterInts = 1 << 16;  // arrival counters at the head of the workspace (shared with the persistent kernel)
constexpr int kGvHeader = kGvCounterInts * 4 + 256;

enum { kGvPlain = 0, kGvRope = 1, kGvSwiglu = 2 };

// One family of kept row blocks: `count` blocks of `keep` rows (rope: rotation pairs, swiglu: channels).
struct GvFam {
  const uint8_t* w;        // rows of MMA row g
  const uint8_t* w2;       // rows of MMA row g + 8 (swiglu: the up matrix; otherwise w)
  const __half* s;  const __half* z;
  const __half* s2; const __half* z2;
  const void* bias;
  void* y;
  int ldy;
  int tile_begin;          // first tile of the family
  int tpb;                 // tiles per kept block
  int keep, count;
  int start, period;       // stored row of block h, row r: start + h * period + r
  int out_base;            // compact output column of block 0, row 0
  int mode;
  int rep;                 // rope: query heads per key-value head
  int head_dim, head_keep; // rope
};

// The activations and the input family.
struct GvQuant {
  const void* x;           // [M][ldx] fp16, compact
  long long ldx;
  // stored channel start + h * period + r (r < keep, h < count) is compact column h * keep + r
  int in_start, in_period, in_keep, in_count;
};

struct GvCfg {
  GvQuant q;
  int M;
  int row_bytes;           // K / 2
  int G;                   // K / 128
  int g_first;             // first visited group (a multiple of GCH)
  int spt;                 // steps per tile: visited groups / GCH
  int tiles_total;
  unsigned U;              // steps of the launch: tiles_total * spt
  unsigned W;              // warps of the launch; warp w takes steps [w * U / W, (w + 1) * U / W)
  int max_slots;           // workspace slots per tile
  int n_fam;
  int xpitch;              // bytes per virtual row of the quantised activations: spt * GCH * 128
  int depth;               // ring slots per warp
  int off_x;               // shared memory: the rings of the warps, then the quantised activations
  GvFam fam[kGvMaxFam];
  int* counters;           // one per tile
  float2* partials;        // [tile][slot][32 lanes]
  const int32_t* idx;
  const int32_t* pos;
  unsigned long long rope_turn[kMaxHalfDim];
};


// asynchronous copies global -> shared (completion is tracked per thread, in groups)
__device__ inline void cpa16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ inline void cpa8(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ inline void cpa_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ inline void cpa_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ inline uint4 lds16(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ inline uint2 lds8(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ inline void gv_mma(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ inline void gv_mma_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ inline float h_lo(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v & 0xffffu))); }
__device__ inline float h_hi(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v >> 16))); }


// stored input channel (a multiple of 4) -> compact activation column, or -1 when the channel is pruned
__device__ inline int gv_compact(const GvQuant& c, int ch) {
  int r = ch - c.in_start;
  if (r < 0) return -1;
  int hh = 0;
  if (c.in_count > 1) {
    hh = r / c.in_period;
    r -= hh * c.in_period;
    if (hh >= c.in_count) return -1;
  }
  return r < c.in_keep ? hh * c.in_keep + r : -1;
}

// bias, rotary embedding or gated product, one rounding, store: lane (g, t) holds the sums of MMA rows g and g + 8
// for batch row t
__device__ inline void gv_store(const GvCfg& c, const GvFam& f, int h, int r0, int g, int m, float va, float vb) {
  __half* y = reinterpret_cast<__half*>(f.y);
  const __half* bias = reinterpret_cast<const __half*>(f.bias);
  if (f.mode == kGvPlain) {
    const int ra = r0 + g, rb = ra + 8;
    const size_t o = (size_t)m * f.ldy + f.out_base + h * f.keep;
    const int sr = f.start + h * f.period;
    if (ra < f.keep) y[o + ra] = __float2half_rn(bias ? va + __half2float(bias[sr + ra]) : va);
    if (rb < f.keep) y[o + rb] = __float2half_rn(bias ? vb + __half2float(bias[sr + rb]) : vb);
  } else if (f.mode == kGvRope) {
    const int cc = r0 + g, half = f.keep;
    if (cc >= half) return;
    if (bias) {
      const int sr = h * f.head_dim + cc;
      va += __half2float(bias[sr]);
      vb += __half2float(bias[sr + (f.head_dim >> 1)]);
    }
    int pidx = c.idx[(h / f.rep) * half + cc];
    pidx = min(max(pidx, 0), (f.head_dim >> 1) - 1);
    float cs, sn;
    rope_cos_sin(c.pos[m], c.rope_turn[pidx], cs, sn);
    const size_t o = (size_t)m * f.ldy + h * f.head_keep + cc;
    y[o] = __float2half_rn(va * cs - vb * sn);
    y[o + half] = __float2half_rn(vb * cs + va * sn);
  } else {
    const int cc = r0 + g;
    if (cc >= f.keep) return;
    // h = g * sigmoid(g) * u, rounded once (the SiLU gate of the MLP paragraph of Section 3.2)
    y[(size_t)m * f.ldy + f.out_base + cc] = __float2half_rn(va / (1.f + __expf(-va)) * vb);
  }
}

// This lane's copy sources in a tile.  A step of a tile is 16 MMA rows x 256 bytes of codes; copy instruction i
// moves MMA rows 2i and 2i + 1, sixteen lanes per row (256 contiguous bytes of a weight row per half-warp), and one
// more instruction moves the scales (lanes 0..15, one MMA row each) and the zero-points (lanes 16..31).
struct GvTile {
  const uint8_t* pw[8];        // codes: MMA row 2i + (lane >> 4), at the first visited group, + (lane & 15) * 16
  const __half* psz;           // scales or zero-points of MMA row lane & 15, at the first visited group
};
// stored row of MMA row r (0..15) of the tile: rows 8..15 are the second member of whatever pairs the mode forms
__device__ inline int gv_row(const GvFam& f, int h, int r0, int r) {
  const int half = r >> 3, rr = r & 7;
  if (f.mode == kGvPlain) return f.start + h * f.period + min(r0 + r, f.keep - 1);
  if (f.mode == kGvRope) return h * f.head_dim + min(r0 + rr, f.keep - 1) + (half ? (f.head_dim >> 1) : 0);
  return f.start + min(r0 + rr, f.keep - 1);
}
__device__ inline void gv_locate(const GvCfg& c, int tile, int lane, GvTile& q) {
  int fi = 0;
  while (fi + 1 < c.n_fam && tile >= c.fam[fi + 1].tile_begin) ++fi;
  const GvFam& f = c.fam[fi];
  const int tl = tile - f.tile_begin;
  const int h = f.count > 1 ? tl / f.tpb : 0;
  const int r0 = (tl - h * f.tpb) * (f.mode == kGvPlain ? 16 : 8);
  const int hi = lane >> 4;
  const size_t col = (size_t)c.g_first * 64 + (size_t)(lane & 15) * 16;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 2 * i + hi;
    q.pw[i] = (r < 8 ? f.w : f.w2) + (size_t)gv_row(f, h, r0, r) * c.row_bytes + col;
  }
  const int r = lane & 15;
  const __half* base = hi ? (r < 8 ? f.z : f.z2) : (r < 8 ? f.s : f.s2);
  q.psz = base + (size_t)gv_row(f, h, r0, r) * c.G + c.g_first;
}

__device__ inline void cpa_wait_dyn(int pending) {      // at most `pending` (0..4) of the latest groups still in flight
  switch (pending) {
    case 0: cpa_wait<0>(); break;
    case 1: cpa_wait<1>(); break;
    case 2: cpa_wait<2>(); break;
    case 3: cpa_wait<3>(); break;
    default: cpa_wait<4>(); break;
  }
}

__global__ void __launch_bounds__(GTH, 1) gemv_kernel(const __grid_constant__ GvCfg c) {
  extern __shared__ __align__(128) unsigned char gsm[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  // the next kernel of the stream may be set up while this one runs
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- this warp's range of the step sequence (32-bit arithmetic: the host checks (U + 1) * W < 2^32)
  const unsigned w = blockIdx.x * GW + warp;
  const bool has_work = w < c.W;
  const unsigned u_begin = has_work ? w * c.U / c.W : 0u, u_end = has_work ? (w + 1) * c.U / c.W : 0u;
  const int n = (int)(u_end - u_begin);
  const int spt = c.spt, GD = c.depth;

  // ---- producer side: the ring of this warp; sixteen lanes copy 256 contiguous bytes of a weight row
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(gsm);
  const uint32_t ring = smem0 + (uint32_t)(warp * GD * kSlotBytes);
  const uint32_t copy_w = ring + (uint32_t)((lane >> 4) * 256 + (((lane & 15) ^ ((lane >> 4) << 2)) * 16));
  const uint32_t copy_s = ring + (uint32_t)(kSlotW + (lane >> 4) * 128 + (lane & 15) * 8);
  int p_tile = (int)(u_begin / (unsigned)spt);
  int p_step = (int)(u_begin - (unsigned)p_tile * (unsigned)spt);
  const int first_step = p_step;                        // where this warp enters its first tile
  GvTile pt;
  if (n > 0) gv_locate(c, p_tile, lane, pt);
  int issued = 0, slot_p = 0;
  auto issue = [&]() {
    const uint32_t dw = copy_w + (uint32_t)(slot_p * kSlotBytes), ds = copy_s + (uint32_t)(slot_p * kSlotBytes);
    const int boff = p_step * (GCH * 64);
#pragma unroll
    for (int i = 0; i < 8; ++i) cpa16(dw + (uint32_t)(i * 512), pt.pw[i] + boff);
    cpa8(ds, pt.psz + p_step * GCH);
    ++issued;
    if (++slot_p == GD) slot_p = 0;
    if (++p_step == spt) {
      p_step = 0;
      ++p_tile;
      if (issued < n) gv_locate(c, p_tile, lane, pt);
    }
  };
  // weights, scales and zero-points are never produced by a preceding kernel: the ring is filled before the
  // dependency wait
  for (int i = 0; i < GD - 1; ++i) {
    if (issued < n) issue();
    cpa_commit();
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");   // activations, outputs, workspace: after the predecessors

  // ---- the block's quantised activations: 16-bit fixed point per (batch row, group), [2M virtual rows][xrow] bytes
  //      in nibble order, then (sum x_i, 2^-e) per (group, batch row)
  const int xrow = c.xpitch + 16;                      // (+16: the eight lanes of a load phase on distinct banks)
  unsigned char* xb = gsm + c.off_x;
  float2* xg = reinterpret_cast<float2*>(xb + (size_t)2 * c.M * xrow);
  {
    const __half* x = reinterpret_cast<const __half*>(c.q.x);
    const int g_count = spt * GCH;
    const int n_units = g_count * c.M * 16;            // a multiple of 32
    constexpr int UN = 4;
    for (int u0 = tid; u0 < n_units; u0 += GTH * UN) {
      uint4 in[UN];
      int mm[UN], lvv[UN];
#pragma unroll
      for (int k = 0; k < UN; ++k) {
        const int u = u0 + k * GTH;
        in[k] = make_uint4(0, 0, 0, 0);
        int lv = u < n_units ? u >> 4 : 0, m = 0;
        while (lv >= g_count) { lv -= g_count; ++m; }
        mm[k] = m; lvv[k] = lv;
        if (u < n_units) {
          const int ch = (c.g_first + lv) * kGroup + 8 * (u & 15);
          const int c0 = gv_compact(c.q, ch), c1 = gv_compact(c.q, ch + 4);
          const __half* xr = x + (size_t)m * c.q.ldx;
          if (c0 >= 0) { const uint2 v = __ldcg(reinterpret_cast<const uint2*>(xr + c0)); in[k].x = v.x; in[k].y = v.y; }
          if (c1 >= 0) { const uint2 v = __ldcg(reinterpret_cast<const uint2*>(xr + c1)); in[k].z = v.x; in[k].w = v.y; }
        }
      }
#pragma unroll
      for (int k = 0; k < UN; ++k) {
        const int u = u0 + k * GTH;
        if (u >= n_units) break;                        // warp-uniform (n_units and GTH are multiples of 32)
        uint2 hi2, lo2;
        int isum;
        float inv_scale;
        quantise16(in[k], hi2, lo2, isum, inv_scale);
        const int u16 = u & 15;
        const int off = lvv[k] * 128 + (u16 >> 2) * 32 + (u16 & 3) * 8;
        *reinterpret_cast<uint2*>(xb + (size_t)(2 * mm[k]) * xrow + off) = hi2;
        *reinterpret_cast<uint2*>(xb + (size_t)(2 * mm[k] + 1) * xrow + off) = lo2;
        if (u16 == 0) xg[lvv[k] * 4 + mm[k]] = make_float2((float)isum, inv_scale);
      }
    }
  }
  __syncthreads();
  if (n == 0) return;

  // ---- consumer side
  const bool xlive = g < 2 * c.M;
  const uint32_t xs_lane = smem0 + (uint32_t)(c.off_x + (xlive ? g : 0) * xrow + t * 32);
  const uint32_t xg_lane = smem0 + (uint32_t)(c.off_x + 2 * c.M * xrow + t * 8);
  // MMA rows g and g + 8 of a slot: 16 bytes at t * 16 of every group (rows of odd parity are stored with the halves
  // of their 128-byte lines exchanged: the two rows of a load phase fall on distinct banks)
  const uint32_t read_w = ring + (uint32_t)(g * 256 + t * 16), read_s = ring + (uint32_t)(kSlotW + g * 8);
  const uint32_t par64 = (uint32_t)((g & 1) * 64);
  int c_tile = (int)(u_begin / (unsigned)spt), c_step = first_step, tile_entry = first_step, slot_c = 0;
  float outA = 0.f, outB = 0.f;

  auto finish_tile = [&](bool whole) {
    if (!whole) {
      // several warps share this tile: park the partial sums; the last to arrive adds them in range order
      const unsigned t0 = (unsigned)c_tile * (unsigned)spt;
      const unsigned first = ((t0 + 1u) * c.W - 1u) / c.U, last = ((t0 + (unsigned)spt) * c.W - 1u) / c.U;
      const int total = (int)(last - first) + 1, mine = (int)(w - first);
      float2* slot0 = c.partials + (size_t)c_tile * c.max_slots * 32 + lane;
      __stcg(slot0 + mine * 32, make_float2(outA, outB));
      __threadfence();
      __syncwarp();
      int is_last = 0;
      if (lane == 0) is_last = atomicAdd(c.counters + c_tile, 1) == total - 1;
      is_last = __shfl_sync(0xffffffffu, is_last, 0);
      if (!is_last) return;
      __threadfence();
      outA = outB = 0.f;
      for (int s2 = 0; s2 < total; ++s2) {
        const float2 v = __ldcg(slot0 + s2 * 32);
        outA += v.x;
        outB += v.y;
      }
      if (lane == 0) c.counters[c_tile] = 0;            // ready for the next call
    }
    if (t < c.M) {
      int fi = 0;
      while (fi + 1 < c.n_fam && c_tile >= c.fam[fi + 1].tile_begin) ++fi;
      const GvFam& f = c.fam[fi];
      const int tl = c_tile - f.tile_begin;
      const int h = f.count > 1 ? tl / f.tpb : 0;
      const int r0 = (tl - h * f.tpb) * (f.mode == kGvPlain ? 16 : 8);
      gv_store(c, f, h, r0, g, t, outA, outB);
    }
  };

  for (int i = 0; i < n; ++i) {
    __syncwarp();                                        // every lane has read the slot that is refilled now
    if (issued < n) issue();
    cpa_commit();
    cpa_wait_dyn(GD - 1);                                // this lane's copies of step i have landed ...
    __syncwarp();                                        // ... and so have the other lanes'
    const uint32_t bw = read_w + (uint32_t)(slot_c * kSlotBytes), bs = read_s + (uint32_t)(slot_c * kSlotBytes);
    const uint2 sav = lds8(bs), zav = lds8(bs + 128), sbv = lds8(bs + 64), zbv = lds8(bs + 192);
    uint4 wa[GCH], wb[GCH], x0[GCH], x1[GCH];
#pragma unroll
    for (int q = 0; q < GCH; ++q) {
      wa[q] = lds16(bw + ((uint32_t)(q * 64) ^ par64));
      wb[q] = lds16(bw + 8 * 256 + ((uint32_t)(q * 64) ^ par64));
      x0[q] = x1[q] = make_uint4(0, 0, 0, 0);
      if (xlive) {
        x0[q] = lds16(xs_lane + (uint32_t)((c_step * GCH + q) * 128));
        x1[q] = lds16(xs_lane + (uint32_t)((c_step * GCH + q) * 128 + 16));
      }
    }
    // the four groups of the step are four independent accumulation chains: word after word, group after group
    int d[GCH][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int q = 0; q < GCH; ++q) {
        const uint32_t w0 = j == 0 ? wa[q].x : j == 1 ? wa[q].y : j == 2 ? wa[q].z : wa[q].w;
        const uint32_t w1 = j == 0 ? wb[q].x : j == 1 ? wb[q].y : j == 2 ? wb[q].z : wb[q].w;
        const uint32_t lo0 = w0 & 0x0f0f0f0fu, hi0 = (w0 >> 4) & 0x0f0f0f0fu;
        const uint32_t lo1 = w1 & 0x0f0f0f0fu, hi1 = (w1 >> 4) & 0x0f0f0f0fu;
        const uint4 xv = (j >> 1) ? x1[q] : x0[q];
        const uint32_t b0 = (j & 1) ? xv.z : xv.x, b1 = (j & 1) ? xv.w : xv.y;
        if (j == 0) gv_mma_first(d[q], lo0, lo1, hi0, hi1, b0, b1);
        else gv_mma(d[q], lo0, lo1, hi0, hi1, b0, b1);
      }
    }
#pragma unroll
    for (int q = 0; q < GCH; ++q) {
      const uint32_t s_a = q < 2 ? sav.x : sav.y, z_a = q < 2 ? zav.x : zav.y;
      const uint32_t s_b = q < 2 ? sbv.x : sbv.y, z_b = q < 2 ? zbv.x : zbv.y;
      const float sa = (q & 1) ? h_hi(s_a) : h_lo(s_a), za = (q & 1) ? h_hi(z_a) : h_lo(z_a);
      const float sb = (q & 1) ? h_hi(s_b) : h_lo(s_b), zb = (q & 1) ? h_hi(z_b) : h_lo(z_b);
      // 256 * (sum q*hi) + (sum q*lo) = sum q*x_i exactly, in integers; one conversion, one rounding
      const float y0 = (float)(d[q][0] * 256 + d[q][1]);
      const float y1 = (float)(d[q][2] * 256 + d[q][3]);
      const uint2 xsb = lds8(xg_lane + (uint32_t)((c_step * GCH + q) * 32));   // (sum x_i, 2^-e) of batch row t
      const float xsum = __uint_as_float(xsb.x), xinv = __uint_as_float(xsb.y);
      outA = fmaf(sa * xinv, fmaf(-za, xsum, y0), outA);
      outB = fmaf(sb * xinv, fmaf(-zb, xsum, y1), outB);
    }
    if (++slot_c == GD) slot_c = 0;
    ++c_step;
    if (c_step == spt || i == n - 1) {
      finish_tile(tile_entry == 0 && c_step == spt);
      outA = outB = 0.f;
      c_step = 0;
      tile_entry = 0;
      ++c_tile;
    }
  }
  cpa_wait<0>();
}

// -------------------------------------------------------------------------------- host side
int gv_sm_count() {
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

size_t gv_align(size_t v) { return (v + 255) & ~(size_t)255; }

// workspace of one launch: header (arrival counters), partial sums [tile][slot][32 lanes], quantised activations
// visited groups of an input family, in whole steps
int gv_group_count(const Fam& a) {
  const int lo = a.start / kGroup / GCH * GCH;
  const int end = a.start + (a.count - 1) * a.period + a.keep;     // exclusive
  return ((end - 1) / kGroup - lo + 1 + GCH - 1) / GCH * GCH;
}
// the quantised activations fit beside rings of at least four slots
bool gv_fits(int M, int g_count) {
  const size_t x_bytes = (size_t)2 * M * (g_count * 128 + 16) + (size_t)g_count * 4 * sizeof(float2);
  return (size_t)GW * 4 * kSlotBytes + x_bytes <= (size_t)kGvSmemMax;
}

struct GvPlan {
  int blocks;
  size_t smem;
  size_t need;
};

// The input family gives the visited groups (whole steps); the tiles give the step sequence and its cut.
int gv_plan(GvCfg* c, const Fam& a, GvPlan* pl) {
  const int lo = a.start / kGroup / GCH * GCH;
  const int end = a.start + (a.count - 1) * a.period + a.keep;     // exclusive
  const int hi = (end - 1) / kGroup;
  const int g_count = (hi - lo + 1 + GCH - 1) / GCH * GCH;
  c->g_first = lo;
  c->spt = g_count / GCH;
  c->xpitch = g_count * 128;
  c->q.in_start = a.start; c->q.in_period = a.period; c->q.in_keep = a.keep; c->q.in_count = a.count;
  if (c->tiles_total < 1 || c->tiles_total > kGvCounterInts) return UNIQL_ERR_UNSUPPORTED;
  const unsigned long long U = (unsigned long long)c->tiles_total * (unsigned)c->spt;
  pl->blocks = gv_sm_count();
  // shared memory: as deep a ring per warp as fits beside the quantised activations
  const size_t x_bytes = (size_t)2 * c->M * (c->xpitch + 16) + (size_t)g_count * 4 * sizeof(float2);
  const int force_depth = opt(kOptGemvDepth);
  int depth = force_depth >= 2 && force_depth <= kGvMaxDepth ? force_depth : kGvMaxDepth;
  while (depth > 2 && (size_t)GW * depth * kSlotBytes + x_bytes > (size_t)kGvSmemMax) --depth;
  if ((size_t)GW * depth * kSlotBytes + x_bytes > (size_t)kGvSmemMax) return UNIQL_ERR_UNSUPPORTED;
  if (depth < 4 && !force_depth) return UNIQL_ERR_UNSUPPORTED;     // too shallow to keep the stream dense
  c->depth = depth;
  c->off_x = GW * depth * kSlotBytes;
  pl->smem = (size_t)c->off_x + x_bytes;
  unsigned long long W = (unsigned long long)pl->blocks * GW;
  if (W > U) {                    // fewer steps than warps: one step per warp (every warp of the cut has work)
    W = U;
    pl->blocks = (int)((W + GW - 1) / GW);
  }
  if ((U + 1) * W >= (1ull << 32)) return UNIQL_ERR_UNSUPPORTED;
  c->U = (unsigned)U;
  c->W = (unsigned)W;
  const unsigned long long per_warp = U / W;
  c->max_slots = per_warp >= 1 ? (int)((unsigned)c->spt / per_warp) + 2 : c->spt;
  if (c->max_slots > c->spt) c->max_slots = c->spt;
  if (c->max_slots < 2) c->max_slots = 2;
  pl->need = gv_align((size_t)kGvHeader + (size_t)c->tiles_total * c->max_slots * 32 * sizeof(float2));
  return UNIQL_OK;
}

int gv_launch(GvCfg* c, const GvPlan& pl, const LaunchCfg& cfg) {
  unsigned char* ws = reinterpret_cast<unsigned char*>(cfg.workspace);
  if (!ws || cfg.ws_bytes < pl.need) return UNIQL_ERR_WORKSPACE;
  c->counters = reinterpret_cast<int*>(ws);
  c->partials = reinterpret_cast<float2*>(ws + kGvHeader);
  {
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return UNIQL_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 0 || dev >= 64 || !done[dev]) {
      if (cudaFuncSetAttribute(gemv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGvSmemMax) != cudaSuccess)
        return UNIQL_ERR_CUDA;
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  const int pdl = opt(kOptPdl);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.stream = cfg.stream;
  lc.attrs = attr;
  lc.numAttrs = pdl ? 1 : 0;
  lc.gridDim = dim3((unsigned)pl.blocks);
  lc.blockDim = dim3(GTH);
  lc.dynamicSmemBytes = pl.smem;
  if (cudaLaunchKernelEx(&lc, gemv_kernel, *c) != cudaSuccess) { cudaGetLastError(); return UNIQL_ERR_CUDA; }
  return UNIQL_OK;
}

}  // namespace

// What the streaming kernel takes: fp16, one to four rows, one input family on 4-channel boundaries, groups per
// stored row a multiple of four, scale / zero-point rows 8-byte aligned.
int gemv_supported(const Params& p) {
  if (p.M < 1 || p.M > 4 || p.dt != UNIQL_F16) return 0;
  if ((p.K % (GCH * kGroup)) != 0) return 0;
  if (p.imap.n_fam != 1) return 0;
  const Fam& a = p.imap.fam[0];
  if ((a.start % 4) || (a.keep % 4) || (a.count > 1 && (a.period % 4))) return 0;
  if ((p.ldx % 4) || (((uintptr_t)p.x) & 7)) return 0;
  int n = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    const JobDev& jb = p.job[j];
    if (jb.pair) return 0;
    if ((((uintptr_t)jb.scales) | ((uintptr_t)jb.zeros)) & 7) return 0;
    if (((uintptr_t)jb.w) & 15) return 0;
    n += jb.rope.enabled ? 1 : jb.omap.n_fam;
  }
  if (!gv_fits(p.M, gv_group_count(a))) return 0;
  return n <= kGvMaxFam;
}

size_t gemv_workspace_bytes(int M, int K, int N_total) {
  // tiles of 8 (rope pairs, gated channels) or 16 rows, one ragged tile per kept block assumed at most per 8 rows
  (void)M;
  const size_t tiles = (size_t)(N_total + 7) / 8 + 2 * kGvMaxFam;
  const size_t spt = (size_t)(K / kGroup + GCH - 1) / GCH + 1;
  const size_t W = (size_t)gv_sm_count() * GW;
  const size_t per_warp = tiles * spt / W;
  size_t slots = per_warp >= 1 ? spt / per_warp + 2 : spt;
  if (slots > spt) slots = spt;
  if (slots < 2) slots = 2;
  return gv_align((size_t)kGvHeader + tiles * slots * 32 * sizeof(float2)) + 256;
}

int launch_gemv(const Params& p, const LaunchCfg& cfg) {
  if (!gemv_supported(p)) return UNIQL_ERR_UNSUPPORTED;
  GvCfg c;
  memset(&c, 0, sizeof(c));
  c.M = p.M; c.row_bytes = p.K / 2; c.G = p.K / kGroup;
  c.q.x = p.x; c.q.ldx = p.ldx;
  c.idx = p.idx; c.pos = p.pos;
  int tiles = 0, n = 0;
  bool any_rope = false;
  for (int j = 0; j < p.n_jobs; ++j) {
    const JobDev& jb = p.job[j];
    if (jb.rope.enabled) {
      GvFam& f = c.fam[n++];
      f.w = f.w2 = jb.w; f.s = f.s2 = jb.scales; f.z = f.z2 = jb.zeros; f.bias = jb.bias; f.y = jb.y; f.ldy = jb.ldy;
      f.tile_begin = tiles; f.keep = jb.rope.head_keep / 2; f.tpb = (f.keep + 7) / 8; f.count = jb.rope.n_heads;
      f.start = 0; f.period = jb.rope.head_dim; f.out_base = 0; f.mode = kGvRope; f.rep = jb.rope.rep;
      f.head_dim = jb.rope.head_dim; f.head_keep = jb.rope.head_keep;
      tiles += f.tpb * f.count;
      any_rope = true;
    } else {
      for (int k = 0; k < jb.omap.n_fam; ++k) {
        const Fam& a = jb.omap.fam[k];
        GvFam& f = c.fam[n++];
        f.w = f.w2 = jb.w; f.s = f.s2 = jb.scales; f.z = f.z2 = jb.zeros; f.bias = jb.bias; f.y = jb.y; f.ldy = jb.ldy;
        f.tile_begin = tiles; f.keep = a.keep; f.tpb = (a.keep + 15) / 16; f.count = a.count;
        f.start = a.start; f.period = a.period; f.out_base = jb.omap.base[k]; f.mode = kGvPlain; f.rep = 1;
        tiles += f.tpb * f.count;
      }
    }
  }
  c.n_fam = n;
  c.tiles_total = tiles;
  if (any_rope) memcpy(c.rope_turn, p.rope_turn, sizeof(c.rope_turn));
  GvPlan pl;
  const int rc = gv_plan(&c, p.imap.fam[0], &pl);
  if (rc) return rc;
  return gv_launch(&c, pl, cfg);
}

// SwiGLU MLP (Section 3.2, MLP paragraph) as two launches of the streaming kernel: gate and up rows of the same
// channel in one lane with silu(g) * u as the epilogue, then the down projection over the leading k_int channels of h.
int gemv_mlp_supported(const MlpDecode& d) {
  if (d.M < 1 || d.M > 4) return 0;
  if ((d.hidden % (GCH * kGroup)) != 0 || (d.inter % (GCH * kGroup)) != 0) return 0;
  if (d.k_int < 4 || d.k_int > d.inter || (d.k_int % 4) != 0) return 0;
  if ((d.ldx % 4) != 0 || (d.ldh % 4) != 0 || d.ldx < d.hidden || d.ldh < d.k_int || d.ldy < d.hidden) return 0;
  if ((((uintptr_t)d.x) | ((uintptr_t)d.h)) & 7) return 0;
  if ((((uintptr_t)d.sg) | ((uintptr_t)d.zg) | ((uintptr_t)d.su) | ((uintptr_t)d.zu) | ((uintptr_t)d.sd) | ((uintptr_t)d.zd)) & 7)
    return 0;
  if ((((uintptr_t)d.wg) | ((uintptr_t)d.wu) | ((uintptr_t)d.wd)) & 15) return 0;
  if (!gv_fits(d.M, gv_group_count(Fam{0, d.hidden, d.hidden, 1})) || !gv_fits(d.M, gv_group_count(Fam{0, d.k_int, d.k_int, 1})))
    return 0;
  return 1;
}

int launch_gemv_mlp(const MlpDecode& d, const LaunchCfg& cfg) {
  if (!gemv_mlp_supported(d)) return UNIQL_ERR_UNSUPPORTED;
  {
    GvCfg c;
    memset(&c, 0, sizeof(c));
    c.M = d.M; c.row_bytes = d.hidden / 2; c.G = d.hidden / kGroup;
    c.q.x = d.x; c.q.ldx = d.ldx;
    GvFam& f = c.fam[0];
    f.w = d.wg; f.s = d.sg; f.z = d.zg; f.w2 = d.wu; f.s2 = d.su; f.z2 = d.zu; f.y = d.h; f.ldy = d.ldh;
    f.tile_begin = 0; f.keep = d.k_int; f.tpb = (d.k_int + 7) / 8; f.count = 1; f.start = 0; f.period = d.inter;
    f.out_base = 0; f.mode = kGvSwiglu; f.rep = 1;
    c.n_fam = 1;
    c.tiles_total = f.tpb;
    GvPlan pl;
    int rc = gv_plan(&c, Fam{0, d.hidden, d.hidden, 1}, &pl);
    if (!rc) rc = gv_launch(&c, pl, cfg);
    if (rc) return rc;
  }
  GvCfg c;
  memset(&c, 0, sizeof(c));
  c.M = d.M; c.row_bytes = d.inter / 2; c.G = d.inter / kGroup;
  c.q.x = d.h; c.q.ldx = d.ldh;
  GvFam& f = c.fam[0];
  f.w = f.w2 = d.wd; f.s = f.s2 = d.sd; f.z = f.z2 = d.zd; f.y = d.y; f.ldy = d.ldy;
  f.tile_begin = 0; f.keep = d.hidden; f.tpb = (d.hidden + 15) / 16; f.count = 1; f.start = 0; f.period = d.hidden;
  f.out_base = 0; f.mode = kGvPlain; f.rep = 1;
  c.n_fam = 1;
  c.tiles_total = f.tpb;
  GvPlan pl;
  const int rc = gv_plan(&c, Fam{0, d.k_int, d.k_int, 1}, &pl);
  if (rc) return rc;
  return gv_launch(&c, pl, cfg);
}

}  // namespace uniql
