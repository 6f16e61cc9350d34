// Decode kernel (M = 1..16) of the pruned 4-bit linear layer, sm_100a.
//
// The decode step streams every retained weight exactly once, so the kernel is built around keeping
// HBM busy: one persistent block per SM whose producer warp keeps a ring of shared-memory stages
// filled by the tensor memory accelerator (cp.async.bulk.tensor boxes of 128 bytes x 64 rows,
// completion on an mbarrier), far ahead of the sixteen consumer warps, and whose epilogue warps
// finish tiles (reduction over the consumer warps, bias, rotary embedding, store) behind them.  No
// role spends registers or issue slots on another role's latency.  On-device pruning (Section 3.4) is expressed in the tensor maps:
// a family of kept channel blocks {start, period, keep, count} is a 3-D tensor (byte in row, row in
// block, block) whose extents stop at the kept rows and at the last visited input group, so pruned
// rows and pruned trailing input channels are out of bounds: never fetched, filled with zeros.
//
// Work decomposition.  A tile is 64 row slots of one kept block, a chunk is 8 quantisation groups
// (1024 input channels, 512 bytes per row).  Every block first takes the same number of whole tiles;
// the (tile, chunk) units of the tiles left over form one chunk-fastest sequence that is cut into equal
// contiguous ranges, one per block (stream-K), so every SM streams the same number of bytes.  A tile
// that is shared by several blocks is finished by the last block to arrive, which adds the parked
// partial sums in a fixed slot order (deterministic, no spinning on other blocks).
//
// Arithmetic.  Inside a stage consumer warp w owns group (w & 7) of the chunk and two 16-row
// sub-tiles.  The packed codes are used as they lie in memory: one LOP3 turns two nibbles of a 32-bit
// word into an fp16 pair (1024+q for a nibble in bits [3:0], 64+q for one in bits [7:4]) and those
// pairs are the A fragments of m16n8k16 tensor-core MMAs whose B fragments are the activations.  The
// contraction index of an MMA is only a label, so the activations are staged once per block in shared
// memory in the order the nibbles come out of a word and no weight byte is ever shuffled.  The
// offsets, the zero-point and the scale are applied once per group and row in fp32:
//     y += s * ( sum_k (o_k + q_k) x_k  -  (sum_k o_k x_k  +  z * sum_k x_k) ),   o_k in {1024, 64}.
// The rotary epilogue (Section 3.2, fused RoPE) needs both members of a rotation pair; in rope mode a
// tile is 32 pairs of one head, first-half members in row slots 0..31 and their partners in 32..63.
//
// Every wait in the kernel is an mbarrier wait with an iteration limit; when one expires the block
// sets the status word of the workspace, lets its copies land and returns.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "quant.cuh"

namespace uniql {
namespace {

constexpr int CW = 16;                  // consumer warps
constexpr int CTH = CW * 32;            // consumer threads
constexpr int EW = 4;                   // epilogue warps
constexpr int ETH = EW * 32;
constexpr int NTH = CTH + 32 + ETH;     // consumers + one producer warp + epilogue warps
constexpr int RB = 64;                  // row slots per tile
constexpr int CG = 8;                   // groups per chunk
constexpr int BOX_COLS = CG / 2;        // 128-byte columns (two groups each) per chunk
constexpr int BOX_BYTES = RB * 128;     // one column of a stage: [RB rows][128 bytes], 128-byte swizzled
constexpr int STAGE_W = BOX_COLS * BOX_BYTES;
constexpr int STAGE_SZ = RB * CG * 2;   // one of the two fp16 arrays [RB][CG]
constexpr int STAGE_BYTES = STAGE_W + 2 * STAGE_SZ;   // a multiple of 1024 (swizzle atom)
constexpr int MAX_STAGES = 6;
constexpr int kCounterInts = 1 << 16;   // arrival counters (one per tile) at the head of the workspace
constexpr int kStatusOff = kCounterInts * 4;   // status word right after the counters
constexpr int kGridSyncOff = kStatusOff + 64;   // the two counters of the barrier between phases
constexpr int kWsHeader = kStatusOff + 256;
constexpr int kMaxKParts = 16;
constexpr int kSmemMax = 227 * 1024;
constexpr int kWaitLimit = 1 << 18;
constexpr int kGridWaitLimit = 1 << 21;   // polls (40 ns apart) of the barrier between the phases of a fused launch
constexpr int BAR_BYTES = 256;
constexpr int kMaxTF = 8;               // (job, family) pairs of one launch

// Division by a divisor the host knows: q = floor(x / d) = umulhi(x, m) with m = floor(2^32 / d) + 1, exact for
// x * d < 2^32 (the host passes m = 0 when that cannot be promised or d = 1: then the plain division is used).
// Integer divisions take about a hundred cycles and several sit on every warp's way to its first unit.
struct FastDiv { unsigned d, m; };
__host__ inline FastDiv fast_div(unsigned d, unsigned long long x_max) {
  FastDiv f;
  f.d = d ? d : 1;
  f.m = (f.d > 1 && x_max * f.d < (1ull << 32)) ? (unsigned)((1ull << 32) / f.d + 1) : 0u;
  return f;
}
__device__ inline int div_by(int x, const FastDiv& f) {
  return f.m ? (int)__umulhi((unsigned)x, f.m) : (f.d == 1 ? x : (int)((unsigned)x / f.d));
}

// One family of kept row blocks of one job: `count` blocks of `keep` rows, tiles of RB rows inside each
// block (rope jobs: blocks are heads, rows are rotation pairs, RB/2 pairs per tile).
struct TileFam {
  int tile_begin;        // first global tile
  int tpb;               // tiles per block
  int keep;              // rows (pairs) per block
  int count;
  int job;
  int start, period;     // stored row of block h, row r: start + h*period + r   (rope: h*head_dim + r)
  int out_base;          // compact output column of block 0, row 0
  int mode;              // kPlain, kNarrow (32 rows x 16 groups), kRope (32 rotation pairs per tile) or
                         // kSwiglu (32 gate rows + 32 up rows)
  int job2;              // kSwiglu: the job of the up projection (`job` is the gate projection)
  FastDiv by_tpb;        // division by tpb
};
enum { kPlain = 0, kRope = 1, kSwiglu = 2, kNarrow = 3 };
__host__ __device__ inline int tile_rows(const TileFam& f) { return f.mode == kPlain ? RB : RB / 2; }

// One matrix product of a launch.  A plain launch has one phase; the fused SwiGLU MLP has two (gate|up,
// then down on the activations the first phase wrote), separated by a grid-wide barrier.
struct Phase {
  const void* x;         // activations [M][ldx]
  long long ldx;
  int K;                 // stored input channels of the phase's matrices
  int start, keep;       // the input family (128-bit staging): head h keeps [start + h*period, +keep)
  int period, count;     // count = 1: a leading block
  int g_total, v_first;  // visited groups and the first of them
  int tile0, tiles;      // global tiles [tile0, tile0 + tiles)
  // the split of the tiles over the blocks, worked out on the host (integer divisions are slow and sit on
  // every warp's way to its first unit): whole tiles per block, left-over tiles, and for a full k-part its
  // groups, chunks per tile and the number of blocks that share the left-over units
  int base, R, gk0, ck0, bt0;
  FastDiv by_ck0, by_bt0;
};

struct DecodeCfg {
  CUtensorMap wmap[kMaxTF];   // packed weights of each family: (byte, row in block, block)
  CUtensorMap wmap_up;        // kSwiglu family: the up projection (wmap[] holds the gate projection)
  TileFam tf[kMaxTF];
  Phase ph[2];
  int n_ph;
  int n_tf;
  int n_kp, n_rp;        // k-parts x blocks per k-part
  int gp;                // visited groups per k-part (the last part may be shorter)
  int g_total;           // visited groups (largest phase)
  int gran;              // groups per scale / zero-point copy granule (2, 4 or 8)
  int cgz;               // groups per chunk: CG, or 2 * CG when the tiles are narrow (all families kNarrow:
                         // row slots 32..63 of a stage then hold the same 32 rows, eight groups further on)
  int stages;
  int tiles_total;
  int x_vec;             // activations can be staged with 128-bit loads
  int max_slots;         // workspace slots per tile
  int off_bar, off_x, xrow, off_xg, off_part, part_bufs;
  int* counters;
  float* partials;
  int* status;
  int* grid_sync;        // two ints: epilogue warps that finished phase 0, blocks that saw all of them
  int grid_wait_limit;   // polls of the barrier between the phases before the block gives up
  // Streamed activations (rows too long to stage whole beside the ring): a small kernel quantises x once
  // into the layout the consumers read, [group][virtual row][128 bytes] plus (integer sum, 2^-e) per (group,
  // batch row), and every stage of the ring carries the eight groups of its unit beside the weights.
  int x_cluster;         // blocks run as clusters of two that share the staging of the activations: each quantises
                         // half of the (row, group) pairs and writes them into both blocks' shared memory
  int x_stream;
  int stage_bytes;       // STAGE_BYTES, plus vr * CG * 128 + 1024 when the activations are streamed
  int vr;                // virtual rows per group in a stage: 8 (up to four batch rows) or 16
  const float2* xg_glob; // [group][8] (integer sum, 2^-e)
  CUtensorMap xmap;      // quantised activations: (byte in line, virtual row, group), 128-byte swizzle
};

// ---------------------------------------------------------------------------------------- PTX helpers
__device__ inline void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ inline void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// more bytes expected in the current phase, without an arrival
__device__ inline void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ inline void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ inline bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// ---- cluster of two (shared staging of the activations)
__device__ inline uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of `addr` (shared memory of this block) in block `rank` of the cluster
__device__ inline uint32_t peer_addr(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ inline void st_peer_v2(uint32_t addr, uint32_t a, uint32_t b) {
  asm volatile("st.shared::cluster.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
__device__ inline void mbar_arrive_peer(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ inline bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit expired or another warp of the block already gave up.
__device__ inline bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < kWaitLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63) == 63 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// One box of a 3-D tensor map into shared memory (no multicast), completion counted on `bar`.
__device__ inline void tma_box3(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// contiguous bytes (a multiple of 16, both sides 16-byte aligned) into shared memory, counted on `bar`
__device__ inline void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ inline void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ inline void cp_async8(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ inline void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ inline void cp_async_arrive_noinc(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// shared-memory loads at [addr + OFF]: the offset is an immediate of the instruction, not an address add
template <int OFF>
__device__ inline uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ inline void lds128_if(uint4& v, uint32_t addr, bool pred) {      // v is left alone when !pred
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%6];\n\t}"
               : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w) : "r"(addr), "r"((uint32_t)pred), "n"(OFF));
}
// line nt * 1024 bytes further on (the index is a constant once the caller's loop is unrolled)
__device__ inline void lds128_line(uint4& v, uint32_t addr, int nt, bool pred) {
  if (nt == 0) lds128_if<0>(v, addr, pred);
  else if (nt == 1) lds128_if<1024>(v, addr, pred);
  else if (nt == 2) lds128_if<2048>(v, addr, pred);
  else lds128_if<3072>(v, addr, pred);
}
template <int OFF>
__device__ inline float4 lds128f(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+%5];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ inline float lds_h(uint32_t addr) {
  unsigned short h;
  asm volatile("ld.shared.u16 %0, [%1+%2];" : "=h"(h) : "r"(addr), "n"(OFF));
  return __half2float(__ushort_as_half(h));
}
// (a & mask) | magic in one LOP3 (truth table 0xEA)
__device__ inline uint32_t and_or(uint32_t a, uint32_t mask, uint32_t magic) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(magic));
  return d;
}
// Eight codes of a 32-bit word as four fp16 pairs: (c0,c4)+1024, (c1,c5)+64, (c2,c6)+1024, (c3,c7)+64.
__device__ inline void cvt_word(uint32_t w, uint32_t (&a)[4]) {
  const uint32_t w8 = w >> 8;
  a[0] = and_or(w, 0x000f000fu, 0x64006400u);
  a[1] = and_or(w, 0x00f000f0u, 0x54005400u);
  a[2] = and_or(w8, 0x000f000fu, 0x64006400u);
  a[3] = and_or(w8, 0x00f000f0u, 0x54005400u);
}
__device__ inline void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                               uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ inline void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the first MMA of a chain: accumulators start at zero (no registers to clear)
__device__ inline void mma_s8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
template <int OFF>
__device__ inline float2 lds64f(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2+%3];" : "=f"(v.x), "=f"(v.y) : "r"(addr), "n"(OFF));
  return v;
}


// stored input channel (a multiple of 8) -> compact activation column, or -1 when the channel is pruned
__device__ inline int compact_channel(const Phase& P, int ch) {
  int r = ch - P.start;
  if (r < 0) return -1;
  int h = 0;
  if (P.count > 1) { h = r / P.period; r -= h * P.period; if (h >= P.count) return -1; }
  return r < P.keep ? h * P.keep + r : -1;
}

// Quantises the activations of one launch once (streamed mode): half-warp (batch row m, visited group lv).
// Rows m >= M of the vr / 2 row slots are written as zeros.
__global__ void __launch_bounds__(256) xquant_kernel(const Phase P, int M, int vr, int g_total, unsigned char* xq,
                                                     float2* xg, int xg_stride) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");            // x may come from the preceding kernel
  const int rows = vr >> 1;
  const int n_units = g_total * rows * 16;
  const __half* x = reinterpret_cast<const __half*>(P.x);
  for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < ((n_units + 31) & ~31); u += gridDim.x * blockDim.x) {
    const int u16 = u & 15, pair = u < n_units ? u >> 4 : 0;
    const int lv = pair / rows, m = pair - lv * rows;
    uint4 in = make_uint4(0, 0, 0, 0);
    if (u < n_units && m < M) {
      const int t0 = compact_channel(P, (P.v_first + lv) * kGroup + 8 * u16);
      if (t0 >= 0) in = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * P.ldx + t0));
    }
    uint2 hi2, lo2;
    int isum;
    float inv_scale;
    quantise16(in, hi2, lo2, isum, inv_scale);
    if (u < n_units) {
      const int off = (u16 >> 2) * 32 + (u16 & 3) * 8;
      *reinterpret_cast<uint2*>(xq + ((size_t)lv * vr + 2 * m) * 128 + off) = hi2;
      *reinterpret_cast<uint2*>(xq + ((size_t)lv * vr + 2 * m + 1) * 128 + off) = lo2;
      if (u16 == 0) xg[lv * xg_stride + m] = make_float2((float)isum, inv_scale);
    }
  }
}

// ---------------------------------------------------------------------------------------- tile geometry
struct TilePos { int fi, h, r0; };
__device__ inline TilePos tile_pos(const DecodeCfg& c, const Params& p, int tg) {
  TilePos q;
  q.fi = 0;
  while (q.fi + 1 < c.n_tf && tg >= c.tf[q.fi + 1].tile_begin) ++q.fi;
  const TileFam& f = c.tf[q.fi];
  const int tl = tg - f.tile_begin;
  q.h = div_by(tl, f.by_tpb);
  q.r0 = (tl - q.h * f.tpb) * tile_rows(f);
  return q;
}
// position of the next tile (tiles are numbered block after block, family after family)
__device__ inline void next_tile(const DecodeCfg& c, const Params& p, TilePos& q) {
  const TileFam& f = c.tf[q.fi];
  q.r0 += tile_rows(f);
  if (q.r0 >= f.keep) {
    q.r0 = 0;
    if (++q.h == f.count) { q.h = 0; ++q.fi; }
  }
}

// The block (of its k-part) whose unit range [U*b/B, U*(b+1)/B) holds unit u: floor(((u + 1) * B - 1) / U), in
// 32-bit integers (the host checks U * B < 2^31).
__device__ inline int owner_of(int u, int B, int U) {
  return (int)(((unsigned)(u + 1) * (unsigned)B - 1u) / (unsigned)U);
}

// bias, rotary embedding on the retained pair, one rounding, store; `get(slot, m)` yields the fp32 sum
template <typename T, typename F>
__device__ inline void store_tile(const Params& p, const TileFam& f, const TilePos& q, int etid, F get) {
  const JobDev& jb = p.job[f.job];
  const T* bias = reinterpret_cast<const T*>(jb.bias);
  T* y = reinterpret_cast<T*>(jb.y);
  if (f.mode == kSwiglu) {
    // slots 0..31 hold the gate rows, slots 32..63 the up rows of the same channels:
    // h = g * sigmoid(g) * u, rounded once (MLP paragraph of Section 3.2, SiLU gate)
    for (int i = etid; i < (RB / 2) * p.M; i += ETH) {
      const int pp = i & (RB / 2 - 1), m = i / (RB / 2);
      const int cc = q.r0 + pp;
      if (cc >= f.keep) continue;
      const float gt = get(pp, m), up = get(pp + RB / 2, m);
      const float hv = gt / (1.f + __expf(-gt)) * up;
      y[(size_t)m * jb.ldy + f.out_base + cc] = DT<T>::from_f(hv);
    }
  } else if (f.mode == kNarrow) {
    for (int i = etid; i < (RB / 2) * p.M; i += ETH) {
      const int pp = i & (RB / 2 - 1), m = i / (RB / 2);
      const int r = q.r0 + pp;
      if (r >= f.keep) continue;
      float v = get(pp, m) + get(pp + RB / 2, m);          // the two halves of the chunk's groups
      if (bias) v += DT<T>::to_f(bias[f.start + q.h * f.period + r]);
      y[(size_t)m * jb.ldy + f.out_base + q.h * f.keep + r] = DT<T>::from_f(v);
    }
  } else if (jb.rope.enabled) {
    const int half = jb.rope.head_keep >> 1;
    for (int i = etid; i < (RB / 2) * p.M; i += ETH) {
      const int pp = i & (RB / 2 - 1), m = i / (RB / 2);
      const int cc = q.r0 + pp;
      if (cc >= half) continue;
      float lo = get(pp, m), hi = get(pp + RB / 2, m);
      if (bias) {
        const int sr = q.h * jb.rope.head_dim + cc;
        lo += DT<T>::to_f(bias[sr]);
        hi += DT<T>::to_f(bias[sr + (jb.rope.head_dim >> 1)]);
      }
      int pidx = p.idx[(q.h / jb.rope.rep) * half + cc];
      pidx = min(max(pidx, 0), (jb.rope.head_dim >> 1) - 1);
      float cs, sn;
      rope_cos_sin(p.pos[m], p.rope_turn[pidx], cs, sn);
      const int oc = q.h * jb.rope.head_keep + cc;
      y[(size_t)m * jb.ldy + oc] = DT<T>::from_f(lo * cs - hi * sn);
      y[(size_t)m * jb.ldy + oc + half] = DT<T>::from_f(hi * cs + lo * sn);
    }
  } else {
    for (int i = etid; i < RB * p.M; i += ETH) {
      const int slot = i & (RB - 1), m = i / RB;
      const int r = q.r0 + slot;
      if (r >= f.keep) continue;
      float v = get(slot, m);
      if (bias) v += DT<T>::to_f(bias[f.start + q.h * f.period + r]);
      y[(size_t)m * jb.ldy + f.out_base + q.h * f.keep + r] = DT<T>::from_f(v);
    }
  }
}

// Blocks that share the R left-over tiles of a k-part with Cq chunks per tile.  Cutting the left-over
// units into n_rp equal ranges (stream-K) balances the bytes but every tile then ends with a hand-over
// between blocks (park, arrival count, reduction by the last block: about the time of three chunks);
// when that costs more than it saves, the left-over tiles are given whole to R blocks instead.
__host__ __device__ inline int tail_blocks(int n_rp, int R, int Cq) {
  const int Ut = R * Cq;
  if (Ut == 0) return 1;
  const bool split = Ut / n_rp + 3 < Cq;
  const int Bt = split ? n_rp : R;
  return Bt < Ut ? Bt : Ut;
}

// ---------------------------------------------------------------------------------------- work split
// Units of one block of k-part `kp`: `base` whole tiles (all chunks) and a contiguous range of the
// chunk-fastest unit sequence of the R tiles that are left over after every block took its share.
struct Work {
  int Ck;            // chunks per tile in this k-part
  int n1;            // units of the whole-tile phase (base * Ck)
  int tile1;         // first whole tile
  int tail_tile0;    // first left-over tile (n_rp * base)
  int tb, te;        // tail unit range [tb, te) in the left-over sequence
  int n_units;
  FastDiv by_ck;     // division by Ck
};
__device__ inline Work block_work(int n_rp, int tile0, int base, int R, int Ck, int Bt_, int rp, const FastDiv& by_ck,
                                  const FastDiv& by_bt) {
  Work w;
  w.Ck = Ck;
  w.by_ck = by_ck;
  // 32-bit arithmetic (64-bit divisions are slow): the host checks n_rp * n_rp * Ck < 2^31
  const unsigned Ut = (unsigned)(R * Ck);
  const unsigned Bt = (unsigned)Bt_;                          // blocks that get tail units
  w.n1 = base * Ck;
  w.tile1 = tile0 + rp * base;
  w.tail_tile0 = tile0 + n_rp * base;
  w.tb = w.te = 0;
  if ((unsigned)rp < Bt) { w.tb = div_by((int)(Ut * (unsigned)rp), by_bt); w.te = div_by((int)(Ut * (unsigned)(rp + 1)), by_bt); }
  w.n_units = w.n1 + (w.te - w.tb);
  return w;
}
// What block (kp, rp) does in one phase.
struct PhaseCtx {
  int Gk;            // groups of this k-part
  int sg_lo;         // its first stored group
  int G;             // groups per stored row
  Work wk;
};
__device__ inline PhaseCtx phase_ctx(const DecodeCfg& c, int ph, int kp, int rp) {
  const Phase& P = c.ph[ph];
  PhaseCtx k;
  const int v_lo = kp * c.gp;                                   // first visit index of this k-part
  k.Gk = min(c.gp, P.g_total - v_lo);
  k.sg_lo = P.v_first + v_lo;
  k.G = P.K / kGroup;
  int Ck = P.ck0, Bt = P.bt0;
  FastDiv by_ck = P.by_ck0, by_bt = P.by_bt0;
  if (k.Gk != P.gk0) {                                          // a shorter last k-part
    Ck = (k.Gk + c.cgz - 1) / c.cgz;
    Bt = tail_blocks(c.n_rp, P.R, Ck);
    by_ck.d = (unsigned)Ck; by_ck.m = 0;
    by_bt.d = (unsigned)Bt; by_bt.m = 0;
  }
  k.wk = block_work(c.n_rp, P.tile0, P.base, P.R, Ck, Bt, rp, by_ck, by_bt);
  return k;
}
// (tile, chunk) of block-local unit i, walked in order.  The share of the left-over tiles comes first:
// its hand-over between blocks (parked sums, arrival count, final reduction by the last block) then
// overlaps the streaming of the whole tiles instead of trailing the kernel.
struct UnitIter {
  int tile, chunk;
  __device__ inline void start(const Work& w) {
    if (w.te > w.tb) { const int t = div_by(w.tb, w.by_ck); tile = w.tail_tile0 + t; chunk = w.tb - t * w.Ck; }
    else { tile = w.tile1; chunk = 0; }
  }
  // returns true when the position jumped (phase switch), i.e. the tile position must be recomputed
  __device__ inline bool advance(const Work& w, int i_next) {
    if (i_next == w.te - w.tb && w.te > w.tb) {
      tile = w.tile1; chunk = 0;
      return true;
    }
    if (++chunk == w.Ck) { chunk = 0; ++tile; }
    return false;
  }
  // unit i is the block's last unit of its tile
  __device__ inline bool tile_end(const Work& w, int i) const {
    return chunk == w.Ck - 1 || i == w.n_units - 1 || i == w.te - w.tb - 1;
  }
};

// ---------------------------------------------------------------------------------------- kernel
// NT == 0: fp16 tensor-core path (MT batch tiles of 8, ONECOL: batch 1).  NT > 0: integer path, NT column
// tiles of the int8 MMA, each holding the high and the low byte of four batch rows.
// NPH: phases (2: the fused SwiGLU MLP, integer path only).  XS: activations streamed through the ring.
// XC: blocks are launched as clusters of two that share the staging of the activations.
template <int MT, bool ONECOL, int NT, int NPH, bool XS, bool XC>
__global__ void __launch_bounds__(NTH, 1) decode_kernel(const __grid_constant__ Params p,
                                                        const __grid_constant__ DecodeCfg c) {
  extern __shared__ unsigned char smem_raw[];
  using T = __half;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // the stage ring starts on a 1024-byte boundary (the swizzle pattern repeats every 1024 bytes)
  const uint32_t raw = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t sbase = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (sbase - raw);
  const int S = c.stages;
  // XS / XC say what this instance can do; whether a launch streams its activations or shares their staging is a
  // flag of the launch (batches of five to eight rows always take the same instance: alternating between two
  // kernel functions costs about 1.5 us per switch)
  // (the instances for nine to sixteen rows each serve one kind of launch only)
  const bool xs_on = XS && (NT == 4 || c.x_stream != 0), xc_on = XC && c.x_cluster != 0;
  // barriers: full[S], empty[S], consumer barrier, (spare), partials full[2] / free[2]; then the abort flag
  const uint32_t bar_full = sbase + c.off_bar, bar_empty = bar_full + 8 * MAX_STAGES;
  const uint32_t bar_cons = bar_full + 16 * MAX_STAGES, bar_epi = bar_cons + 8;
  const uint32_t bar_pfull = bar_cons + 16, bar_pfree = bar_cons + 32;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + c.off_bar + 16 * MAX_STAGES + 48);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(bar_full + 8 * s, 33);      // one expect_tx arrival + 32 copy-completion arrivals
      mbar_init(bar_empty + 8 * s, CW);
    }
    mbar_init(bar_cons, CW);
    mbar_init(bar_epi, xc_on ? 2 * CW : EW);        // shared staging: the consumer warps of both blocks arrive
    for (int b = 0; b < 2; ++b) { mbar_init(bar_pfull + 8 * b, CW); mbar_init(bar_pfree + 8 * b, EW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // shared staging: every thread of the pair arrives at the cluster barrier once its block's barriers exist; the
  // consumer warps wait for it before they first touch the other block's shared memory
  if (xc_on) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  int kp = 0, rp = (int)blockIdx.x;
  if (c.n_kp > 1) { kp = rp / c.n_rp; rp -= kp * c.n_rp; }
  // Programmatic dependent launch: the next kernel of the stream may be set up while this one runs (its
  // blocks still need this block's resources, so they start as blocks here exit) ...
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const PhaseCtx pc0 = phase_ctx(c, 0, kp, rp);
  if (NPH == 1 && pc0.wk.n_units == 0) return;

  // ======================================================================================= producer
  // The ring runs on across phases: the weights of the next phase are fetched while the grid-wide barrier
  // between the phases is still being crossed (weights, scales and zero-points are never produced in here).
  if (warp == CW) {
    int it = 0, s = 0;
    uint32_t ring_parity = 1;      // parity of the previous use of ring position s
    bool ok = true;
    // Streamed activations are written by the kernel launched just before this one.  The weights of the first
    // fill of the ring do not wait for it: their stages are armed with the weight bytes only, and once the ring
    // is full (or the block's units are all issued) the producer waits for the predecessor and sends the
    // activations of those stages after them, with the arrival the stages' barriers still lack.
    bool x_waited = !xs_on;
    int x_lv0[MAX_STAGES];
    auto send_x = [&](int stage, int lv0) {                          // lane 31: arrival + the unit's activations
      const uint32_t full = bar_full + 8 * stage;
      const uint32_t st = sbase + (uint32_t)stage * (uint32_t)c.stage_bytes;
      mbar_expect_tx(full, (uint32_t)(c.vr * CG * 128 + CG * 64 * MT));
      tma_box3(st + STAGE_BYTES, &c.xmap, 0, 0, lv0, full);
      bulk_copy(st + STAGE_BYTES + (uint32_t)(c.vr * CG * 128), c.xg_glob + (size_t)lv0 * 8 * MT, CG * 64 * MT, full);
    };
    auto flush_x = [&](int n_issued) {                               // after the first min(S, units) stages
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (lane == 31)
        for (int j = 0; j < n_issued; ++j) send_x(j, x_lv0[j]);
      __syncwarp();
      x_waited = true;
    };
    for (int ph = 0; ph < NPH && ok; ++ph) {
      const PhaseCtx pc = (NPH == 1 || ph == 0) ? pc0 : phase_ctx(c, ph, kp, rp);
      const Work& wk = pc.wk;
      const int Gk = pc.Gk, sg_lo = pc.sg_lo, G = pc.G;
      if (wk.n_units == 0) continue;
      UnitIter ui;
      ui.start(wk);
      int tile_prev = -1;
      bool jumped = true;
      TilePos q = {0, 0, 0};
      int mode = kPlain;
      const __half* srow[2] = {nullptr, nullptr};
      const __half* zrow[2] = {nullptr, nullptr};
      for (int iu = 0; iu < wk.n_units; ++iu, ++it) {
        if (it >= S) ok = mbar_wait(bar_empty + 8 * s, ring_parity, abort_flag);
        if (!ok) break;
        const bool new_tile = ui.tile != tile_prev;
        if (new_tile) {
          if (jumped) q = tile_pos(c, p, ui.tile); else next_tile(c, p, q);
          jumped = false;
          mode = c.tf[q.fi].mode;
          tile_prev = ui.tile;
        }
        // (the rows of scales and zero-points of a new tile are worked out after its first weight boxes are on
        //  their way: they need several more dependent reads of the kernel parameters)
        auto setup_rows = [&]() {
          const TileFam& f = c.tf[q.fi];
#pragma unroll
          for (int r2 = 0; r2 < 2; ++r2) {
            const JobDev& jb = p.job[(mode == kSwiglu && r2) ? f.job2 : f.job];
            const int slot = lane + 32 * r2;
            int sr = -1;
            if (mode == kRope) {
              const int cc = q.r0 + lane;
              if (cc < f.keep) sr = q.h * jb.rope.head_dim + r2 * (jb.rope.head_dim >> 1) + cc;
            } else if (mode == kSwiglu) {
              const int cc = q.r0 + lane;
              if (cc < f.keep) sr = f.start + cc;
            } else if (mode == kNarrow) {
              const int r = q.r0 + lane;
              if (r < f.keep) sr = f.start + q.h * f.period + r;
            } else {
              const int r = q.r0 + slot;
              if (r < f.keep) sr = f.start + q.h * f.period + r;
            }
            const int gsh = mode == kNarrow ? r2 * CG : 0;       // the second half of a narrow chunk
            srow[r2] = sr >= 0 ? jb.scales + (size_t)sr * G + sg_lo + gsh : nullptr;
            zrow[r2] = sr >= 0 ? jb.zeros + (size_t)sr * G + sg_lo + gsh : nullptr;
          }
        };
        const int chunk = ui.chunk;
        const int ng_all = min(c.cgz, Gk - chunk * c.cgz);  // visited groups of the unit
        const int ng = min(CG, ng_all), ng2 = ng_all - ng;  // ... in row slots 0..31 (all 64 unless narrow) / 32..63
        const int nb = (ng + 1) >> 1, nb2 = (ng2 + 1) >> 1; // 128-byte columns with a visited group
        const uint32_t full = bar_full + 8 * s;
        const uint32_t st = sbase + (uint32_t)s * (xs_on ? (uint32_t)c.stage_bytes : (uint32_t)STAGE_BYTES);
        const uint32_t wbytes = mode == kNarrow ? (uint32_t)((nb + nb2) * (BOX_BYTES / 2)) : (uint32_t)(nb * BOX_BYTES);
        if (xs_on) {
          if (lane == 0) mbar_expect_tx_only(full, wbytes);          // the arrival comes with the activations
          if (!x_waited) x_lv0[s] = chunk * CG;                      // (one k-part, wide tiles; s == it here)
        } else if (lane == 0) {
          mbar_expect_tx(full, wbytes);
        }
        __syncwarp();
        if (xs_on && x_waited && lane == 31) send_x(s, chunk * CG);
        if (lane < nb) {
          const int xb = (sg_lo + chunk * c.cgz + 2 * lane) * 64;    // byte in the weight row
          const uint32_t dst = st + (uint32_t)lane * BOX_BYTES;
          if (mode == kNarrow) {
            tma_box3(dst, &c.wmap[q.fi], xb, q.r0, q.h, full);
            if (lane < nb2) tma_box3(dst + (RB / 2) * 128, &c.wmap[q.fi], xb + CG * 64, q.r0, q.h, full);
          } else if (mode == kRope) {
            tma_box3(dst, &c.wmap[q.fi], xb, q.r0, 2 * q.h, full);
            tma_box3(dst + (RB / 2) * 128, &c.wmap[q.fi], xb, q.r0, 2 * q.h + 1, full);
          } else if (mode == kSwiglu) {
            tma_box3(dst, &c.wmap[q.fi], xb, q.r0, 0, full);
            tma_box3(dst + (RB / 2) * 128, &c.wmap_up, xb, q.r0, 0, full);
          } else {
            tma_box3(dst, &c.wmap[q.fi], xb, q.r0, q.h, full);
          }
        }
        if (new_tile) setup_rows();
#pragma unroll
        for (int r2 = 0; r2 < 2; ++r2) {
          const int ngr = (mode == kNarrow && r2) ? ng2 : ng;      // groups of this half of the row slots
          if (srow[r2] && ngr > 0) {
            const int slot = lane + 32 * r2;
            const uint32_t sd = st + STAGE_W + slot * (CG * 2), zd = sd + STAGE_SZ;
            const __half* sp = srow[r2] + chunk * c.cgz;
            const __half* zp = zrow[r2] + chunk * c.cgz;
            if (c.gran == 8) {
              cp_async16(sd, sp); cp_async16(zd, zp);
            } else if (c.gran == 4) {
              for (int g4 = 0; g4 < ngr; g4 += 4) { cp_async8(sd + g4 * 2, sp + g4); cp_async8(zd + g4 * 2, zp + g4); }
            } else {
              for (int g2 = 0; g2 < ngr; g2 += 2) { cp_async4(sd + g2 * 2, sp + g2); cp_async4(zd + g2 * 2, zp + g2); }
            }
          }
        }
        cp_async_arrive_noinc(full);
        if (iu + 1 < wk.n_units && ui.advance(wk, iu + 1)) jumped = true;
        if (++s == S) { s = 0; ring_parity ^= 1; }
        if (xs_on && !x_waited && it + 1 == S) flush_x(S);
      }
      if (xs_on && !x_waited) flush_x(it);                              // fewer units than stages
    }
    if (!ok) {
      // let the copies of the stages that are still armed land before the block goes away
      const int first = it > S ? it - S : 0;
      for (int j = first; j < it; ++j) {
        const uint32_t full = bar_full + 8 * (j % S);
        for (int i = 0; i < kWaitLimit && !mbar_try_wait(full, (j / S) & 1); ++i) {}
      }
      if (lane == 0) atomicExch(c.status, UNIQL_ERR_TIMEOUT);
    }
    return;
  }

  float* part = reinterpret_cast<float*>(smem + c.off_part);
  const int RM = RB * p.M;
  const int part_stride = CG * RM;           // floats per partial buffer

  // ======================================================================================= epilogue
  // Finishes the block's tiles in order, behind the consumers: sums the eight parked group partials of
  // every (row slot, batch row), then stores the tile, or parks the sum for the block that finishes it.
  if (warp > CW) {
    const int etid = tid - (CW + 1) * 32;
    auto give_up = [&]() { if (lane == 0) atomicExch(c.status, UNIQL_ERR_TIMEOUT); };
    int tiles_done = 0;
    // ... and this kernel may have been started before its predecessor finished: outputs, workspace, bias,
    // positions and indices are touched only after the predecessor is complete (the producer warp does not
    // wait: weights, scales and zero-points are not produced by a preceding decode launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int ph = 0; ph < NPH; ++ph) {
      const PhaseCtx pc = (NPH == 1 || ph == 0) ? pc0 : phase_ctx(c, ph, kp, rp);
      const Work& wk = pc.wk;
      const Phase& P = c.ph[ph];
      UnitIter ui;
      TilePos q = {0, 0, 0};
      if (wk.n_units > 0) {
        ui.start(wk);
        q = tile_pos(c, p, ui.tile);
      }
      for (int i = 0; i < wk.n_units; ++i) {
        const bool tile_end = ui.tile_end(wk, i);
        if (tile_end) {
          const int buf = c.part_bufs > 1 ? (tiles_done & 1) : 0;
          const int use = c.part_bufs > 1 ? (tiles_done >> 1) : tiles_done;
          if (!mbar_wait(bar_pfull + 8 * buf, use & 1, abort_flag)) { give_up(); return; }
          const float* pr = part + buf * part_stride;
          auto local_sum = [&](int slot, int m) -> float {
            float v = 0.f;
#pragma unroll
            for (int q8 = 0; q8 < CG; ++q8) v += pr[q8 * RM + m * RB + slot];
            return v;
          };
          const int tile = ui.tile;
          const TileFam& f = c.tf[q.fi];
          // how many blocks (over all k-parts) work on this tile, and which of them am I
          int total = 0, my_slot = 0;
          const bool tail = tile >= wk.tail_tile0;
          if (c.n_kp == 1 && !tail) {
            total = 1;
          } else {
            const int R = P.R;
            for (int q2 = 0; q2 < c.n_kp; ++q2) {
              int n_here = 1, first = rp;                      // a whole tile: one block per k-part
              if (tail) {
                const int Gq = min(c.gp, P.g_total - q2 * c.gp);
                const int Cq = Gq == P.gk0 ? P.ck0 : (Gq + c.cgz - 1) / c.cgz;
                const int Ut = R * Cq;
                const int Bt = Gq == P.gk0 ? P.bt0 : tail_blocks(c.n_rp, R, Cq);
                const int t0 = (tile - wk.tail_tile0) * Cq;
                first = owner_of(t0, Bt, Ut);
                n_here = owner_of(t0 + Cq - 1, Bt, Ut) - first + 1;
              }
              if (q2 == kp) my_slot = total + (rp - first);
              total += n_here;
            }
          }
          if (total == 1) {
            store_tile<T>(p, f, q, etid, local_sum);
          } else {
            // Hand-over without block-wide barriers: every epilogue warp owns the same output items in all
            // blocks (item i belongs to warp (i / 32) % EW), parks the sums of its items, counts its own
            // arrival, and the last warp of its kind to arrive finishes its items.
            float* tile_ws = c.partials + (size_t)tile * c.max_slots * RM;
            float* mine = tile_ws + (size_t)my_slot * RM;
            if (f.mode != kPlain) {
              for (int j = etid; j < (RB / 2) * p.M; j += ETH) {
                const int pp = j & (RB / 2 - 1), m = j / (RB / 2);
                __stcg(mine + m * RB + pp, local_sum(pp, m));
                __stcg(mine + m * RB + pp + RB / 2, local_sum(pp + RB / 2, m));
              }
            } else {
              for (int j = etid; j < RM; j += ETH) __stcg(mine + j, local_sum(j & (RB - 1), j / RB));
            }
            __threadfence();
            __syncwarp();
            int last_w = 0;
            int* cnt = c.counters + tile * EW + (warp - CW - 1);
            if (lane == 0) {
              last_w = atomicAdd(cnt, 1) == total - 1;
              __threadfence();
            }
            last_w = __shfl_sync(0xffffffffu, last_w, 0);
            if (last_w) {
              auto global_sum = [&](int slot, int m) -> float {
                float v = 0.f;
                for (int s2 = 0; s2 < total; ++s2) v += __ldcg(tile_ws + (size_t)s2 * RM + m * RB + slot);
                return v;
              };
              store_tile<T>(p, f, q, etid, global_sum);
              if (lane == 0) *cnt = 0;                   // ready for the next call
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_pfree + 8 * buf);
          ++tiles_done;
        }
        if (i + 1 < wk.n_units) {
          const int tile_before = ui.tile;
          if (ui.advance(wk, i + 1)) q = tile_pos(c, p, ui.tile);
          else if (ui.tile != tile_before) next_tile(c, p, q);
        }
      }
      if (NPH > 1 && ph + 1 < NPH) {
        // this warp's outputs of the phase (tiles it stored, sums it parked) are complete and visible:
        // count it at the grid-wide barrier the consumers of every block wait on before the next phase
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(c.grid_sync, 1);
      }
    }
    return;
  }

  // ======================================================================================= consumers
  const int ctid = tid;                    // 0..CTH-1
  const int g = lane >> 2, t = lane & 3;
  const int kpw = warp & 7, rg = warp >> 3;
  // MMA row g of a sub-tile is row slot pg: lanes g = 2i and 2i+1 get slots that differ in bit 2, so that
  // under the 128-byte swizzle the eight lanes of a shared-memory load phase touch eight distinct 16-byte columns
  const int pg = (g >> 1) | ((g & 1) << 2);
  // group of the chunk this warp works on: narrow tiles put eight more groups of the same rows in slots 32..63
  const int g_first = c.cgz > CG ? rg * CG + kpw : kpw;
  uint32_t cons_parity = 0;
  auto give_up = [&]() { if (lane == 0) atomicExch(c.status, UNIQL_ERR_TIMEOUT); };
  auto consumer_sync = [&]() -> bool {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_cons);
    const bool ok = mbar_wait(bar_cons, cons_parity, abort_flag);
    cons_parity ^= 1;
    if (!ok) give_up();
    return ok;
  };

  // ---- stage activations: permuted into nibble order, zero where the channel is pruned; per group and
  //      batch row the two sums the offset / zero-point correction needs, stored negated
  auto stage_x = [&](int ph, const PhaseCtx& pc) -> bool {
    const Phase& P = c.ph[ph];
    const Work& wk = pc.wk;
    const int Gk = pc.Gk, sg_lo = pc.sg_lo;
    const T* x = reinterpret_cast<const T*>(P.x);
    const long long ldx = P.ldx;
    // stored channel (a multiple of 8) -> compact activation column, or -1 when the channel is pruned
    const int m_start = P.start, m_keep = P.keep;
    const bool m_heads = P.count > 1;
    auto compact_of = [&](int ch) -> int {
      if (m_heads) return compact_channel(P, ch);
      const int r = ch - m_start;
      return (r >= 0 && r < m_keep) ? r : -1;
    };
    // activations a previous phase of this launch wrote are read past the non-coherent cache
    auto load16 = [&](const T* ptr) -> uint4 {
      return (NPH > 1 && ph > 0) ? __ldcg(reinterpret_cast<const uint4*>(ptr)) : __ldg(reinterpret_cast<const uint4*>(ptr));
    };
    const int row_units = c.xrow / 16;
    uint4* xs = reinterpret_cast<uint4*>(smem + c.off_x);
    float2* xg = reinterpret_cast<float2*>(smem + c.off_xg);
    // Groups this block needs: all visited groups, or, for a block that only holds a short run of left-over
    // units (K-heavy matrices), the chunks of that run.
    int ch0 = 0, n_ch = wk.Ck;
    if (wk.n1 == 0 && wk.te - wk.tb < wk.Ck) { ch0 = wk.tb % wk.Ck; n_ch = wk.te - wk.tb; }
    const int cgz = c.cgz, cg_sh = c.cgz > CG ? 4 : 3;
    const int Gn = n_ch * cgz;
    // batch row of (row, group) pair number `pair` = pair / Gn, without the division (at most 15 steps)
    auto row_of = [&](int pair) { int m = 0; while (pair >= Gn) { pair -= Gn; ++m; } return m; };
    auto needed_group = [&](int gn) { int ch = ch0 + (gn >> cg_sh); if (ch >= wk.Ck) ch -= wk.Ck; return (ch << cg_sh) + (gn & (cgz - 1)); };
    if (NT == 0) {          // (the integer path writes every entry it later reads)
      for (int i = ctid; i < Gk * 8 * MT; i += CTH) xg[i] = make_float2(0.f, 0.f);
      if (!consumer_sync()) return false;
    }
    if (NT > 0) {
      // Integer path.  Per (batch row, group) the activations become 16-bit fixed point, x_i = rint(x * 2^e)
      // with 2^e the largest power of two that keeps the group's maximum at or below 32639 (so that the high
      // byte of x_i + 128 stays a signed byte; exact for every element within a factor 8..16 of the maximum,
      // since fp16 carries 11 bits; smaller elements are rounded to 2^-15..2^-14 of the maximum).
      // x_i = 256 * hi + lo with both bytes signed; the bytes go to two "virtual"
      // batch rows (columns 2m and 2m+1 of the int8 MMA), in the order the nibbles leave a weight word:
      // even codes in the first register of a word's pair, odd codes in the second.
      // Shared staging (clusters of two): this block quantises the pairs of its own parity and writes them into
      // both blocks' shared memory (same layout, same offsets); the other block does the same for the rest.
      const bool xc = xc_on;
      const int crank = xc ? (int)cluster_rank() : 0, csh = xc ? 1 : 0;
      const int n_pairs = Gn * p.M;
      const int n_units = ((n_pairs - crank + csh) >> csh) * 16;     // units of this block's pairs
      unsigned char* xb = smem + c.off_x;
      uint32_t px = 0, pxg = 0;                                      // the other block's x and xg regions
      if (xc) {
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // its barriers exist
        px = peer_addr(sbase + (uint32_t)c.off_x, (uint32_t)(crank ^ 1));
        pxg = peer_addr(sbase + (uint32_t)c.off_xg, (uint32_t)(crank ^ 1));
      }
      constexpr int UN = 4;
      for (int u0 = ctid; u0 < ((n_units + 31) & ~31); u0 += CTH * UN) {
        uint4 in[UN];
#pragma unroll
        for (int q4 = 0; q4 < UN; ++q4) {
          const int u = u0 + q4 * CTH;
          in[q4] = make_uint4(0, 0, 0, 0);
          if (u < n_units) {
            const int pair = ((u >> 4) << csh) + crank, m = row_of(pair), lv = needed_group(pair - m * Gn);
            const int t0 = compact_of((sg_lo + lv) * kGroup + 8 * (u & 15));
            if (lv < Gk && t0 >= 0) in[q4] = load16(x + (size_t)m * ldx + t0);
          }
        }
#pragma unroll
        for (int q4 = 0; q4 < UN; ++q4) {
          const int u = u0 + q4 * CTH;
          if (u >= ((n_units + 31) & ~31)) break;                  // warp-uniform
          const int u16 = u & 15, pair = u < n_units ? ((u >> 4) << csh) + crank : 0;
          const int m = row_of(pair), lv = needed_group(pair - m * Gn);
          const bool in_range = u < n_units && lv < Gk;
          uint2 hi2, lo2;
          int isum;
          float inv_scale;
          quantise16(in[q4], hi2, lo2, isum, inv_scale);
          if (in_range) {
            // word j of lane quarter c' (u16 = c'*4 + j): 8 bytes at c'*32 + j*8 of the group's 128 bytes
            const int off = lv * 128 + (u16 >> 2) * 32 + (u16 & 3) * 8;
            *reinterpret_cast<uint2*>(xb + (size_t)(2 * m) * c.xrow + off) = hi2;
            *reinterpret_cast<uint2*>(xb + (size_t)(2 * m + 1) * c.xrow + off) = lo2;
            if (u16 == 0) xg[lv * 8 * MT + m] = make_float2((float)isum, inv_scale);
            if (xc) {
              st_peer_v2(px + (uint32_t)((2 * m) * c.xrow + off), hi2.x, hi2.y);
              st_peer_v2(px + (uint32_t)((2 * m + 1) * c.xrow + off), lo2.x, lo2.y);
              if (u16 == 0) st_peer_v2(pxg + (uint32_t)((lv * 8 * MT + m) * 8), (uint32_t)__float_as_int((float)isum),
                                       (uint32_t)__float_as_int(inv_scale));
            }
          }
        }
      }
      if (xc) {
        // both halves are in place once the sixteen consumer warps of each block have arrived at this block's
        // barrier (bounded wait; the other block cannot leave before it has seen this block's arrivals, and this
        // block writes nothing into it after them)
        __syncwarp();
        if (lane == 0) {
          asm volatile("fence.acq_rel.cluster;" ::: "memory");
          mbar_arrive(bar_epi);
          mbar_arrive_peer(peer_addr(bar_epi, (uint32_t)(crank ^ 1)));
        }
        bool ok = false;
        for (int i = 0; i < kWaitLimit && !ok; ++i) {
          ok = mbar_try_wait_cluster(bar_epi, 0);
          if (!ok && (i & 63) == 63 && *abort_flag) break;
        }
        if (!ok) { *abort_flag = 1; give_up(); return false; }
        return true;
      }
    } else if (c.x_vec) {
      const int n_units = Gn * p.M * 16;
      constexpr int UN = 4;                                        // loads in flight per thread
      for (int u0 = ctid; u0 < ((n_units + 31) & ~31); u0 += CTH * UN) {   // whole warps stay in the shuffles
        uint4 in[UN];
#pragma unroll
        for (int q4 = 0; q4 < UN; ++q4) {
          const int u = u0 + q4 * CTH;
          in[q4] = make_uint4(0, 0, 0, 0);
          if (u < n_units) {
            const int pair = u >> 4, m = row_of(pair), lv = needed_group(pair - m * Gn);
            const int t0 = compact_of((sg_lo + lv) * kGroup + 8 * (u & 15));
            if (lv < Gk && t0 >= 0) in[q4] = load16(x + (size_t)m * ldx + t0);
          }
        }
#pragma unroll
        for (int q4 = 0; q4 < UN; ++q4) {
          const int u = u0 + q4 * CTH;
          if (u >= ((n_units + 31) & ~31)) break;                  // warp-uniform
          const int u16 = u & 15, pair = u < n_units ? u >> 4 : 0;
          const int m = row_of(pair), lv = needed_group(pair - m * Gn);
          const bool in_range = u < n_units && lv < Gk;
          uint4 o;
          o.x = __byte_perm(in[q4].x, in[q4].z, 0x5410); o.y = __byte_perm(in[q4].x, in[q4].z, 0x7632);
          o.z = __byte_perm(in[q4].y, in[q4].w, 0x5410); o.w = __byte_perm(in[q4].y, in[q4].w, 0x7632);
          // the 16 bytes of lane quarter c', word j of a group sit at byte j*64 + c'*16; u16 = c'*4 + j
          if (in_range) xs[m * row_units + lv * 16 + (u16 & 3) * 4 + (u16 >> 2)] = o;
          const __half2* h2 = reinterpret_cast<const __half2*>(&in[q4]);
          float se = 0.f, so = 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) { const float2 f = __half22float2(h2[i]); se += f.x; so += f.y; }
#pragma unroll
          for (int o2 = 8; o2 >= 1; o2 >>= 1) {
            se += __shfl_xor_sync(0xffffffffu, se, o2);
            so += __shfl_xor_sync(0xffffffffu, so, o2);
          }
          if (in_range && u16 == 0) xg[lv * 8 * MT + m] = make_float2(-(se + so), -(1024.f * se + 64.f * so));
        }
      }
    } else {
      T* xh = reinterpret_cast<T*>(smem + c.off_x);
      const int n_pairs = Gk * p.M;
      for (int pair = warp; pair < n_pairs; pair += CW) {
        const int m = pair / Gk, lv = pair - m * Gk;
        const int kbase = (sg_lo + lv) * kGroup;
        float se = 0.f, so = 0.f;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int i = lane + 32 * q4;
          T val = __float2half_rn(0.f);
          const int tt = map_stored_to_compact(p.imap, kbase + i);
          if (tt >= 0) val = x[(size_t)m * ldx + tt];
          const int ccq = i >> 5, j = (i & 31) >> 3, e = i & 7;
          xh[(m * row_units + lv * 16 + j * 4 + ccq) * 8 + 2 * (e & 3) + (e >> 2)] = val;
          if (i & 1) so += __half2float(val); else se += __half2float(val);
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) {
          se += __shfl_xor_sync(0xffffffffu, se, o2);
          so += __shfl_xor_sync(0xffffffffu, so, o2);
        }
        if (lane == 0) xg[lv * 8 * MT + m] = make_float2(-(se + so), -(1024.f * se + 64.f * so));
      }
    }
    if (!consumer_sync()) return false;
    return true;
  };
  asm volatile("griddepcontrol.wait;" ::: "memory");       // the activations may come from the preceding kernel

  if constexpr (NT > 0) {
    // ===================================================================== consumers, integer path
    // Per weight word: low nibbles and high nibbles as bytes (AND, SHR, AND) are the A fragments of one
    // m16n8k32 int8 MMA for two weight rows; B holds the activation bytes.  Column 2m of the MMA sums
    // q * hi, column 2m+1 sums q * lo: both land in the same lane, 256 * d_hi + d_lo is sum q * x_i exactly.
    uint32_t xaddr8[NT];
    bool xlive8[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int v = g + 8 * nt;                        // virtual batch row: 2m (high bytes), 2m+1 (low bytes)
      xlive8[nt] = v < 2 * p.M;
      xaddr8[nt] = sbase + c.off_x + (uint32_t)((xlive8[nt] ? v : 0) * c.xrow + t * 32);
    }
    const uint32_t xgaddr8 = sbase + c.off_xg + (uint32_t)(t * 8);           // batch row m = t + 4 nt
    // streamed activations: line (group kpw, virtual row v) of the stage, its 16-byte chunks XOR-ed with v & 7
    const bool xstream = xs_on;
    uint32_t xs0[NT], xs1[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int v = g + 8 * nt;
      const uint32_t line = (uint32_t)(STAGE_BYTES + (kpw * c.vr + (v < c.vr ? v : 0)) * 128);
      xs0[nt] = line + (uint32_t)(((2 * t) ^ (v & 7)) * 16);
      xs1[nt] = line + (uint32_t)(((2 * t + 1) ^ (v & 7)) * 16);
    }
    const uint32_t xsg = (uint32_t)(STAGE_BYTES + c.vr * CG * 128 + kpw * 64 * MT + t * 8);
    const uint32_t wl_off = (uint32_t)((kpw >> 1) * BOX_BYTES + (rg * 32 + pg) * 128 + ((((kpw & 1) * 4 + t) ^ pg) * 16));
    const uint32_t sl_off = (uint32_t)(STAGE_W + (rg * 32 + pg) * (CG * 2) + kpw * 2);
    float out8[2][NT][2];
#pragma unroll
    for (int sub = 0; sub < 2; ++sub)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) out8[sub][nt][0] = out8[sub][nt][1] = 0.f;
    uint4 xr8[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) xr8[nt][0] = xr8[nt][1] = make_uint4(0, 0, 0, 0);
    int tiles_done = 0;
    int s = 0;
    uint32_t ring_parity = 0;
    for (int ph = 0; ph < NPH; ++ph) {
    const PhaseCtx pc = (NPH == 1 || ph == 0) ? pc0 : phase_ctx(c, ph, kp, rp);
    const Work& wk = pc.wk;
    const int Gk = pc.Gk;
    if (NPH > 1 && ph > 0) {
      // Grid-wide barrier: the activations of this phase are complete once every epilogue warp of the grid
      // has counted itself in.  One thread polls (bounded), the consumer barrier releases the others; the
      // last block to see the full count clears both counters for the next launch.
      if (warp == 0 && lane == 0) {
        const int target = (int)gridDim.x * EW;
        bool seen = false;
        for (int i = 0; i < c.grid_wait_limit && !seen; ++i) {
          int v;
          asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(c.grid_sync) : "memory");
          seen = v >= target;
          if (!seen) {
            if (*abort_flag) break;
            __nanosleep(40);
          }
        }
        if (seen) {
          __threadfence();
          if (atomicAdd(c.grid_sync + 1, 1) == (int)gridDim.x - 1) {
            c.grid_sync[0] = 0;
            c.grid_sync[1] = 0;
            __threadfence();
          }
        } else {
          // the wait ran out: the whole block leaves (the other roles see the flag in their own bounded waits)
          *abort_flag = 1;
          atomicExch(c.status, UNIQL_ERR_TIMEOUT);
        }
      }
      if (!consumer_sync() || *abort_flag) return;
    }
    if (wk.n_units == 0) continue;
    if (!xstream && !stage_x(ph, pc)) return;
    UnitIter ui;
    ui.start(wk);
    for (int i = 0; i < wk.n_units; ++i) {
      if (!mbar_try_wait(bar_full + 8 * s, ring_parity) && !mbar_wait(bar_full + 8 * s, ring_parity, abort_flag)) {
        give_up();
        return;
      }
      const int gi = ui.chunk * c.cgz + g_first;
      if (gi < Gk) {
        const uint32_t st = sbase + (uint32_t)s * (xs_on ? (uint32_t)c.stage_bytes : (uint32_t)STAGE_BYTES);
        const uint32_t wp = st + wl_off, sp = st + sl_off;
        if constexpr (NT <= 1) {
        uint4 wa[2], wb[2];
        wa[0] = lds128<0>(wp);
        wb[0] = lds128<8 * 128>(wp);
        wa[1] = lds128<16 * 128>(wp);
        wb[1] = lds128<24 * 128>(wp);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const uint32_t xa = xaddr8[nt] + (uint32_t)(gi * 128);
          lds128_if<0>(xr8[nt][0], xstream ? st + xs0[nt] : xa, xlive8[nt]);
          lds128_if<0>(xr8[nt][1], xstream ? st + xs1[nt] : xa + 16, xlive8[nt]);
        }
        float sc[2][2], zp[2][2];
        sc[0][0] = lds_h<0>(sp);
        sc[0][1] = lds_h<8 * CG * 2>(sp);
        sc[1][0] = lds_h<16 * CG * 2>(sp);
        sc[1][1] = lds_h<24 * CG * 2>(sp);
        zp[0][0] = lds_h<STAGE_SZ>(sp);
        zp[0][1] = lds_h<STAGE_SZ + 8 * CG * 2>(sp);
        zp[1][0] = lds_h<STAGE_SZ + 16 * CG * 2>(sp);
        zp[1][1] = lds_h<STAGE_SZ + 24 * CG * 2>(sp);
        int d[2][NT][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            const uint32_t w0 = j == 0 ? wa[sub].x : j == 1 ? wa[sub].y : j == 2 ? wa[sub].z : wa[sub].w;
            const uint32_t w1 = j == 0 ? wb[sub].x : j == 1 ? wb[sub].y : j == 2 ? wb[sub].z : wb[sub].w;
            const uint32_t lo0 = w0 & 0x0f0f0f0fu, hi0 = (w0 >> 4) & 0x0f0f0f0fu;
            const uint32_t lo1 = w1 & 0x0f0f0f0fu, hi1 = (w1 >> 4) & 0x0f0f0f0fu;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const uint4 xv = xr8[nt][j >> 1];
              const uint32_t b0 = (j & 1) ? xv.z : xv.x, b1 = (j & 1) ? xv.w : xv.y;
              if (j == 0) mma_s8_first(d[sub][nt], lo0, lo1, hi0, hi1, b0, b1);
              else mma_s8(d[sub][nt], lo0, lo1, hi0, hi1, b0, b1);
            }
          }
        }
        const uint32_t xga = xstream ? st + xsg : xgaddr8 + (uint32_t)(gi * 8 * MT * 8);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float2 xs = nt == 0 ? lds64f<0>(xga) : nt == 1 ? lds64f<32>(xga) : nt == 2 ? lds64f<64>(xga) : lds64f<96>(xga);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            // 256 * (sum q*hi) + (sum q*lo) = sum q*x_i exactly, in integers; one conversion, one rounding
            const float y0 = (float)(d[sub][nt][0] * 256 + d[sub][nt][1]);
            const float y1 = (float)(d[sub][nt][2] * 256 + d[sub][nt][3]);
            out8[sub][nt][0] = fmaf(sc[sub][0] * xs.y, fmaf(-zp[sub][0], xs.x, y0), out8[sub][nt][0]);
            out8[sub][nt][1] = fmaf(sc[sub][1] * xs.y, fmaf(-zp[sub][1], xs.x, y1), out8[sub][nt][1]);
          }
        }
        } else {
          // Two or four column tiles (five to sixteen rows): the two halves of the warp's 32 weight rows one after
          // the other; the nibbles of a half are split once (16 words) and each column tile then runs its chain of
          // four MMAs and its scaling on its own, so that 4 accumulators and the activation bytes of one tile are
          // live at a time (all four tiles at once need more registers than a thread of this block can have:
          // 284 bytes of spills inside this loop; with two tiles this order measured 3-4 % faster than all
          // accumulators at once, with one tile slightly slower).
          const uint32_t xga = xs_on ? st + xsg : xgaddr8 + (uint32_t)(gi * 8 * MT * 8);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            uint32_t lo0[4], lo1[4], hi0[4], hi1[4];
            {
              const uint4 wa = sub == 0 ? lds128<0>(wp) : lds128<16 * 128>(wp);
              const uint4 wb = sub == 0 ? lds128<8 * 128>(wp) : lds128<24 * 128>(wp);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint32_t w0 = j == 0 ? wa.x : j == 1 ? wa.y : j == 2 ? wa.z : wa.w;
                const uint32_t w1 = j == 0 ? wb.x : j == 1 ? wb.y : j == 2 ? wb.z : wb.w;
                lo0[j] = w0 & 0x0f0f0f0fu; hi0[j] = (w0 >> 4) & 0x0f0f0f0fu;
                lo1[j] = w1 & 0x0f0f0f0fu; hi1[j] = (w1 >> 4) & 0x0f0f0f0fu;
              }
            }
            const float sc0 = sub == 0 ? lds_h<0>(sp) : lds_h<16 * CG * 2>(sp);
            const float sc1 = sub == 0 ? lds_h<8 * CG * 2>(sp) : lds_h<24 * CG * 2>(sp);
            const float zp0 = sub == 0 ? lds_h<STAGE_SZ>(sp) : lds_h<STAGE_SZ + 16 * CG * 2>(sp);
            const float zp1 = sub == 0 ? lds_h<STAGE_SZ + 8 * CG * 2>(sp) : lds_h<STAGE_SZ + 24 * CG * 2>(sp);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              uint4 xa = make_uint4(0, 0, 0, 0), xb = make_uint4(0, 0, 0, 0);
              if (xs_on) {
                lds128_line(xa, st + xs0[0], nt, true);
                lds128_line(xb, st + xs1[0], nt, true);
              } else {
                lds128_if<0>(xa, xaddr8[nt] + (uint32_t)(gi * 128), xlive8[nt]);
                lds128_if<16>(xb, xaddr8[nt] + (uint32_t)(gi * 128), xlive8[nt]);
              }
              const float2 xs = nt == 0 ? lds64f<0>(xga) : nt == 1 ? lds64f<32>(xga) : nt == 2 ? lds64f<64>(xga) : lds64f<96>(xga);
              int d[4];
              mma_s8_first(d, lo0[0], lo1[0], hi0[0], hi1[0], xa.x, xa.y);
              mma_s8(d, lo0[1], lo1[1], hi0[1], hi1[1], xa.z, xa.w);
              mma_s8(d, lo0[2], lo1[2], hi0[2], hi1[2], xb.x, xb.y);
              mma_s8(d, lo0[3], lo1[3], hi0[3], hi1[3], xb.z, xb.w);
              const float y0 = (float)(d[0] * 256 + d[1]);
              const float y1 = (float)(d[2] * 256 + d[3]);
              out8[sub][nt][0] = fmaf(sc0 * xs.y, fmaf(-zp0, xs.x, y0), out8[sub][nt][0]);
              out8[sub][nt][1] = fmaf(sc1 * xs.y, fmaf(-zp1, xs.x, y1), out8[sub][nt][1]);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * s);
      if (++s == S) { s = 0; ring_parity ^= 1; }
      if (ui.tile_end(wk, i)) {
        const int buf = c.part_bufs > 1 ? (tiles_done & 1) : 0;
        const int use = c.part_bufs > 1 ? (tiles_done >> 1) : tiles_done;
        if (use > 0 && !mbar_wait(bar_pfree + 8 * buf, (use - 1) & 1, abort_flag)) { give_up(); return; }
        float* pb = part + buf * part_stride + kpw * RM;
#pragma unroll
        for (int sub = 0; sub < 2; ++sub)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int m = t + 4 * nt;
            if (m < p.M) {
              pb[m * RB + rg * 32 + sub * 16 + pg] = out8[sub][nt][0];
              pb[m * RB + rg * 32 + sub * 16 + pg + 8] = out8[sub][nt][1];
            }
            out8[sub][nt][0] = out8[sub][nt][1] = 0.f;
          }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_pfull + 8 * buf);
        ++tiles_done;
      }
      if (i + 1 < wk.n_units) ui.advance(wk, i + 1);
    }
    }   // phases
    return;
  }

  // ===================================================================== consumers, fp16 path (one phase)
  const PhaseCtx& pc = pc0;
  const Work& wk = pc.wk;
  const int Gk = pc.Gk;
  if (!stage_x(0, pc)) return;
  // per-lane shared-memory addresses
  uint32_t xaddr[MT];
  bool xlive[MT];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int m = g + 8 * mt;
    xlive[mt] = m < p.M;
    xaddr[mt] = sbase + c.off_x + (uint32_t)((xlive[mt] ? m : 0) * c.xrow + t * 16);
  }
  const uint32_t xgaddr = sbase + c.off_xg + (uint32_t)(2 * t * 8);
  const uint32_t wl_off = (uint32_t)((kpw >> 1) * BOX_BYTES + (rg * 32 + pg) * 128 + ((((kpw & 1) * 4 + t) ^ pg) * 16));
  const uint32_t sl_off = (uint32_t)(STAGE_W + (rg * 32 + pg) * (CG * 2) + kpw * 2);

  float out[2][MT][4];
#pragma unroll
  for (int sub = 0; sub < 2; ++sub)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int i = 0; i < 4; ++i) out[sub][mt][i] = 0.f;

  UnitIter ui;
  ui.start(wk);
  int tiles_done = 0;
  int s = 0;                 // ring position and the parity of its current use
  uint32_t ring_parity = 0;
  uint4 xr[MT][4];           // B fragments; lanes whose batch row does not exist keep zeros
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < 4; ++j) xr[mt][j] = make_uint4(0, 0, 0, 0);
  for (int i = 0; i < wk.n_units; ++i) {
    if (!mbar_try_wait(bar_full + 8 * s, ring_parity) && !mbar_wait(bar_full + 8 * s, ring_parity, abort_flag)) {
      give_up();
      return;
    }
    const int gi = ui.chunk * c.cgz + g_first;
    if (gi < Gk) {
      const uint32_t st = sbase + (uint32_t)s * (uint32_t)STAGE_BYTES;
      const uint32_t wp = st + wl_off, sp = st + sl_off;
      uint4 wa[2], wb[2];
      wa[0] = lds128<0>(wp);
      wb[0] = lds128<8 * 128>(wp);
      wa[1] = lds128<16 * 128>(wp);
      wb[1] = lds128<24 * 128>(wp);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const uint32_t xa = xaddr[mt] + (uint32_t)(gi * 256);
        lds128_if<0>(xr[mt][0], xa, xlive[mt]);
        lds128_if<64>(xr[mt][1], xa, xlive[mt]);
        lds128_if<128>(xr[mt][2], xa, xlive[mt]);
        lds128_if<192>(xr[mt][3], xa, xlive[mt]);
      }
      float acc[2][MT][4];
      float sc[2][2];
      sc[0][0] = lds_h<0>(sp);
      sc[0][1] = lds_h<8 * CG * 2>(sp);
      sc[1][0] = lds_h<16 * CG * 2>(sp);
      sc[1][1] = lds_h<24 * CG * 2>(sp);
      float zp[2][2];
      zp[0][0] = lds_h<STAGE_SZ>(sp);
      zp[0][1] = lds_h<STAGE_SZ + 8 * CG * 2>(sp);
      zp[1][0] = lds_h<STAGE_SZ + 16 * CG * 2>(sp);
      zp[1][1] = lds_h<STAGE_SZ + 24 * CG * 2>(sp);
      const uint32_t xga = xgaddr + (uint32_t)(gi * 8 * MT * 8);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        // (-sum x, -sum o x) of batch rows 2t, 2t+1 (+8 mt)
        const float4 xc = mt == 0 ? lds128f<0>(xga) : lds128f<64>(xga);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          acc[sub][mt][0] = fmaf(zp[sub][0], xc.x, xc.y);
          acc[sub][mt][2] = fmaf(zp[sub][1], xc.x, xc.y);
          acc[sub][mt][1] = ONECOL ? 0.f : fmaf(zp[sub][0], xc.z, xc.w);
          acc[sub][mt][3] = ONECOL ? 0.f : fmaf(zp[sub][1], xc.z, xc.w);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          const uint32_t w0 = j == 0 ? wa[sub].x : j == 1 ? wa[sub].y : j == 2 ? wa[sub].z : wa[sub].w;
          const uint32_t w1 = j == 0 ? wb[sub].x : j == 1 ? wb[sub].y : j == 2 ? wb[sub].z : wb[sub].w;
          uint32_t a[4], b[4];
          cvt_word(w0, a);
          cvt_word(w1, b);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            mma_f16(acc[sub][mt], a[0], b[0], a[1], b[1], xr[mt][j].x, xr[mt][j].y);
            mma_f16(acc[sub][mt], a[2], b[2], a[3], b[3], xr[mt][j].z, xr[mt][j].w);
          }
        }
      }
#pragma unroll
      for (int sub = 0; sub < 2; ++sub)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          out[sub][mt][0] = fmaf(sc[sub][0], acc[sub][mt][0], out[sub][mt][0]);
          out[sub][mt][2] = fmaf(sc[sub][1], acc[sub][mt][2], out[sub][mt][2]);
          if (!ONECOL) {
            out[sub][mt][1] = fmaf(sc[sub][0], acc[sub][mt][1], out[sub][mt][1]);
            out[sub][mt][3] = fmaf(sc[sub][1], acc[sub][mt][3], out[sub][mt][3]);
          }
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * s);
    if (++s == S) { s = 0; ring_parity ^= 1; }

    const bool tile_end = ui.tile_end(wk, i);
    if (tile_end) {
      // ---- park this warp's partial sums for the epilogue warps: part[buf][group slot kpw][m][row slot]
      const int buf = c.part_bufs > 1 ? (tiles_done & 1) : 0;
      const int use = c.part_bufs > 1 ? (tiles_done >> 1) : tiles_done;
      if (use > 0 && !mbar_wait(bar_pfree + 8 * buf, (use - 1) & 1, abort_flag)) { give_up(); return; }
      float* pb = part + buf * part_stride + kpw * RM;
#pragma unroll
      for (int sub = 0; sub < 2; ++sub)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int e = 0; e < (ONECOL ? 1 : 2); ++e) {
            const int m = 2 * t + e + 8 * mt;
            if (m < p.M) {
              pb[m * RB + rg * 32 + sub * 16 + pg] = out[sub][mt][e];
              pb[m * RB + rg * 32 + sub * 16 + pg + 8] = out[sub][mt][2 + e];
            }
          }
#pragma unroll
      for (int sub = 0; sub < 2; ++sub)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int i2 = 0; i2 < 4; ++i2) out[sub][mt][i2] = 0.f;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_pfull + 8 * buf);
      ++tiles_done;
    }
    if (i + 1 < wk.n_units) ui.advance(wk, i + 1);
  }
}

// -------------------------------------------------------------------------------- host side
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

int round_up(int a, int b) { return (a + b - 1) / b * b; }

int copy_granule(int G) { return (G % 8 == 0) ? 8 : (G % 4 == 0) ? 4 : 2; }

// number of (job, family) pairs of a launch
int count_tile_fams(const Params& p) {
  int n = 0;
  for (int j = 0; j < p.n_jobs; ++j) n += p.job[j].rope.enabled ? 1 : p.job[j].omap.n_fam;
  return n;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link-time dependency on libcuda).
EncodeTiledFn encoder() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      cudaGetLastError();
  });
  return fn;
}

// Packed rows of one family as a 3-D byte tensor (byte in row, row in block, block), 128-byte swizzled boxes.
int encode_family(CUtensorMap* tm, const uint8_t* base, int K, int x_extent, int keep, int count, int row_stride_rows,
                  int box_rows) {
  EncodeTiledFn enc = encoder();
  if (!enc) return UNIQL_ERR_CUDA;
  const cuuint64_t dims[3] = {(cuuint64_t)x_extent, (cuuint64_t)keep, (cuuint64_t)count};
  const cuuint64_t strides[2] = {(cuuint64_t)(K / 2), (cuuint64_t)row_stride_rows * (cuuint64_t)(K / 2)};
  const cuuint32_t box[3] = {128, (cuuint32_t)box_rows, 1};
  const cuuint32_t es[3] = {1, 1, 1};
  const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t*>(base), dims, strides, box, es,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? UNIQL_OK : UNIQL_ERR_CUDA;
}

// Shared-memory plan for a given split; returns the total size in bytes (with the alignment slack).
size_t plan_smem(DecodeCfg* c, int M, int MT, int gp, int stages, int part_bufs, bool i8) {
  size_t off = (size_t)stages * STAGE_BYTES;
  c->off_bar = (int)off;
  off += BAR_BYTES;
  // fp16 path: one row of gp*256 bytes per batch row (+64: lane pairs on distinct banks);
  // integer path: two rows (high and low bytes) of gp*128 bytes per batch row (+16)
  c->xrow = i8 ? gp * 128 + 16 : gp * 256 + 64;
  c->off_x = (int)off;
  off += (size_t)M * (i8 ? 2 : 1) * c->xrow;
  off = (off + 15) & ~(size_t)15;
  c->off_xg = (int)off;
  off += (size_t)gp * 8 * MT * 8;
  c->off_part = (int)off;
  off += (size_t)part_bufs * CG * RB * M * 4;
  c->stages = stages;
  c->part_bufs = part_bufs;
  return off + 1024;
}

// Worst-case number of workspace slots a tile needs for a given split: one per k-part for a whole tile,
// one per block that shares it for a left-over tile.
int slots_needed(int tiles, int g_total, int gp, int n_rp, int cgz) {
  int total = 0;
  const int base = tiles / n_rp;
  const long R = tiles - (long)base * n_rp;
  for (int v = 0; v < g_total; v += gp) {
    const long Gq = (g_total - v) < gp ? (g_total - v) : gp;
    const long Cq = (Gq + cgz - 1) / cgz;
    const long Ut = R * Cq;
    if (Ut == 0) { total += 1; continue; }
    const long Bt = tail_blocks(n_rp, (int)R, (int)Cq);
    const long per_block = Ut / Bt;           // >= 1
    total += (int)((Cq + per_block - 1) / per_block) + 1;
  }
  return total;
}

// Time of the slowest block, in units (one stage of the ring), for `tiles` tiles of Ck units over n_rp blocks:
// whole tiles, then the left-over tiles either cut into equal ranges (plus the hand-over) or given whole.
long schedule_cost(long tiles, long Ck, long n_rp) {
  const long base = tiles / n_rp, R = tiles - base * n_rp;
  if (R == 0) return base * Ck;
  const bool split = R * Ck / n_rp + 3 < Ck;                 // the rule of tail_blocks()
  return base * Ck + (split ? (R * Ck + n_rp - 1) / n_rp + 3 : Ck);
}

// the host's part of the work split of one phase (see Phase)
void fill_split(const DecodeCfg& c, Phase* P) {
  P->base = P->tiles / c.n_rp;
  P->R = P->tiles - P->base * c.n_rp;
  P->gk0 = P->g_total < c.gp ? P->g_total : c.gp;
  P->ck0 = (P->gk0 + c.cgz - 1) / c.cgz;
  P->bt0 = tail_blocks(c.n_rp, P->R, P->ck0);
  const unsigned long long ut = (unsigned long long)P->R * P->ck0;
  P->by_ck0 = fast_div((unsigned)P->ck0, ut);
  P->by_bt0 = fast_div((unsigned)P->bt0, ut * (unsigned long long)c.n_rp);
}

template <int MT, bool ONECOL, int NT, int NPH, bool XS = false, bool XC = false>
int launch_t(const Params& p, const DecodeCfg& c, size_t smem, cudaStream_t stream) {
  auto kern = decode_kernel<MT, ONECOL, NT, NPH, XS, XC>;
  {
    // the shared-memory limit of this instance is raised once per device (the call costs about a microsecond)
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return UNIQL_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 0 || dev >= 64 || !done[dev]) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax) != cudaSuccess)
        return UNIQL_ERR_CUDA;
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3(c.n_kp * c.n_rp);
  lc.blockDim = dim3(NTH);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[2];
  lc.attrs = attr;
  if (NPH > 1) {
    // the blocks of a fused launch wait on one another: all of them must be resident at once
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    lc.numAttrs = 1;
  } else {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.numAttrs = opt(kOptPdl) ? 1 : 0;
  }
  DecodeCfg cc = c;
  const bool as_clusters = XC && c.x_cluster != 0;
  if (as_clusters) {
    // clusters of two (shared staging): only when every pair can be resident at once, else plain blocks
    attr[lc.numAttrs].id = cudaLaunchAttributeClusterDimension;
    attr[lc.numAttrs].val.clusterDim.x = 2;
    attr[lc.numAttrs].val.clusterDim.y = 1;
    attr[lc.numAttrs].val.clusterDim.z = 1;
    ++lc.numAttrs;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, kern, &lc) != cudaSuccess || n_clusters * 2 < (int)lc.gridDim.x) {
      cudaGetLastError();
      return UNIQL_ERR_UNSUPPORTED;        // the caller launches plain blocks instead
    }
  }
  if (cudaLaunchKernelEx(&lc, kern, p, cc) == cudaSuccess) return UNIQL_OK;
  cudaGetLastError();
  return as_clusters ? UNIQL_ERR_UNSUPPORTED : UNIQL_ERR_CUDA;
}

// Visited groups of the input map: from the first to the last 128-channel group that holds a retained
// channel, widened to the copy granule (gaps between families are visited with zero activations).
void visited_range(const ChanMap& m, int gran, int* first, int* total) {
  int lo = m.fam[0].start / kGroup, hi = 0;
  for (int f = 0; f < m.n_fam; ++f) {
    const Fam& a = m.fam[f];
    const int end = a.start + (a.count - 1) * a.period + a.keep;   // exclusive
    const int last = (end - 1) / kGroup;
    if (last > hi) hi = last;
  }
  lo = lo / gran * gran;
  *first = lo;
  *total = hi - lo + 1;
}

// Split of the visited groups into k-parts and the shared-memory plan: as few k-parts as let the staged
// activations fit beside a deep enough ring of stages.  Returns 0 when nothing fits.
size_t plan_split(DecodeCfg* c, int M, int g_total, int gran, bool i8) {
  const int MT = M <= 8 ? 1 : 2;
  const int part_bufs = M <= 8 ? 2 : 1;
  int n_kp = opt(kOptDecodeKp);
  const int stages = opt(kOptDecodeStages);
  const int want = (stages >= 2 && stages <= MAX_STAGES) ? stages : 4;
  size_t smem = 0;
  bool fits = false;
  if (n_kp >= 1) {
    if (n_kp > kMaxKParts) n_kp = kMaxKParts;
    const int gp = round_up((g_total + n_kp - 1) / n_kp, gran);
    for (int s = want; s >= 2 && !fits; --s) {
      smem = plan_smem(c, M, MT, gp, s, part_bufs, i8);
      fits = smem <= (size_t)kSmemMax;
    }
    c->gp = gp;
  } else {
    for (n_kp = 1; n_kp <= kMaxKParts && !fits; ++n_kp)
      for (int s = want; s >= 3 && !fits; --s) {
        const int gp = round_up((g_total + n_kp - 1) / n_kp, gran);
        smem = plan_smem(c, M, MT, gp, s, part_bufs, i8);
        fits = smem <= (size_t)kSmemMax;
        c->gp = gp;
      }
  }
  if (!fits) return 0;
  c->g_total = g_total;
  c->gran = gran;
  c->n_kp = (g_total + c->gp - 1) / c->gp;
  int n_rp = opt(kOptDecodeRp);
  if (n_rp < 1) n_rp = sm_count() / c->n_kp;
  if (n_rp < 1) n_rp = 1;
  c->n_rp = n_rp;
  // the kernel cuts the left-over units with 32-bit products of at most n_rp * n_rp * (chunks per tile)
  if ((long long)n_rp * n_rp * ((c->gp + CG - 1) / CG) >= (1ll << 31)) return 0;
  return smem;
}

// Shared-memory plan with streamed activations: no staged copy of x, every stage carries the unit's eight
// groups of quantised activations.  One k-part.  Returns 0 when nothing fits.
size_t plan_stream(DecodeCfg* c, int M, int g_total, int gran) {
  c->vr = M <= 4 ? 8 : (M <= 8 ? 16 : 32);
  c->stage_bytes = STAGE_BYTES + c->vr * CG * 128 + 1024;
  const int tries[6][2] = {{4, 2}, {4, 1}, {3, 2}, {3, 1}, {2, 2}, {2, 1}};
  for (int i = 0; i < 6; ++i) {
    const int stages = tries[i][0], part_bufs = tries[i][1];
    size_t off = (size_t)stages * c->stage_bytes;
    c->off_bar = (int)off;
    off += BAR_BYTES;
    c->off_x = c->off_xg = (int)off;
    c->xrow = 0;
    c->off_part = (int)off;
    off += (size_t)part_bufs * CG * RB * M * 4;
    if (off + 1024 > (size_t)kSmemMax) continue;
    c->stages = stages;
    c->part_bufs = part_bufs;
    c->gp = round_up(g_total, gran);
    c->g_total = g_total;
    c->gran = gran;
    c->n_kp = 1;
    int n_rp = opt(kOptDecodeRp);
    if (n_rp < 1) n_rp = sm_count();
    c->n_rp = n_rp;
    if ((long long)n_rp * n_rp * ((c->gp + CG - 1) / CG) >= (1ll << 31)) return 0;
    return off + 1024;
  }
  return 0;
}

// Streamed activations, host side.  The quantised copy sits in the workspace behind the partial sums:
// [groups, padded to whole chunks][vr virtual rows][128 bytes], then one (sum, 1 / scale) pair per group and
// batch-row slot (8 slots up to eight rows, 16 above).
struct StreamWs { size_t xq_off, xg_off; int g_pad, slots; };
size_t stream_need(const DecodeCfg& c, int M, int g_total, size_t need, StreamWs* o) {
  o->g_pad = round_up(g_total, CG);
  o->slots = M <= 8 ? 8 : 16;
  o->xq_off = (need + 255) & ~(size_t)255;
  o->xg_off = o->xq_off + (size_t)o->g_pad * c.vr * 128;
  return o->xg_off + (size_t)o->g_pad * 8 * o->slots;
}
// The tensor map over the quantised copy, and the small kernel in front that writes it (once per launch).
int stream_setup(DecodeCfg& c, const Phase& P, int M, int g_total, unsigned char* ws, const StreamWs& o,
                 cudaStream_t stream) {
  EncodeTiledFn enc = encoder();
  if (!enc) return UNIQL_ERR_CUDA;
  const cuuint64_t dims[3] = {128, (cuuint64_t)c.vr, (cuuint64_t)o.g_pad};
  const cuuint64_t strides[2] = {128, (cuuint64_t)c.vr * 128};
  const cuuint32_t box[3] = {128, (cuuint32_t)c.vr, (cuuint32_t)CG};
  const cuuint32_t es[3] = {1, 1, 1};
  if (enc(&c.xmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, ws + o.xq_off, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return UNIQL_ERR_CUDA;
  c.xg_glob = reinterpret_cast<const float2*>(ws + o.xg_off);
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  const int units = g_total * (c.vr / 2) * 16;
  lc.gridDim = dim3((units + 255) / 256);
  lc.blockDim = dim3(256);
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = opt(kOptPdl) ? 1 : 0;
  if (cudaLaunchKernelEx(&lc, xquant_kernel, P, M, c.vr, g_total, ws + o.xq_off,
                         reinterpret_cast<float2*>(ws + o.xg_off), o.slots) != cudaSuccess) {
    cudaGetLastError();
    return UNIQL_ERR_CUDA;
  }
  return UNIQL_OK;
}

}  // namespace

// Nine to sixteen rows in one launch: the activations of so many rows never fit beside the ring, so they are
// streamed through it; the integer path only (option "decode_split_batch" 2, the default).
int decode_streams_batch(const Params& p) {
  return p.M > 8 && p.M <= 16 && opt(kOptDecodeSplitBatch) == 2 && opt(kOptDecodeI8) != 0 &&
         opt(kOptDecodeXstream) != 0 && decode_integer_path(p);
}

int decode_supported(const Params& p) {
  if (p.M < 1 || p.M > 16) return 0;
  if (p.dt != UNIQL_F16) return 0;
  if ((p.K % (2 * kGroup)) != 0) return 0;
  if (count_tile_fams(p) > kMaxTF) return 0;
  const int gran = copy_granule(p.K / kGroup);
  for (int j = 0; j < p.n_jobs; ++j) {
    // scale / zero-point rows are copied in granules of 2, 4 or 8 fp16 values
    if (((uintptr_t)p.job[j].scales | (uintptr_t)p.job[j].zeros) & (uintptr_t)(gran * 2 - 1)) return 0;
  }
  return 1;
}

// The integer path of this kernel applies: one input family, everything on 8-channel boundaries, 128-bit loads.
int decode_integer_path(const Params& p) {
  return p.imap.n_fam == 1 && (p.imap.fam[0].start % 8) == 0 && (p.imap.fam[0].keep % 8) == 0 &&
         (p.imap.fam[0].count == 1 || (p.imap.fam[0].period % 8) == 0) && (p.ldx % 8) == 0 &&
         ((((uintptr_t)p.x) & 15) == 0);
}

size_t decode_workspace_bytes(int M, int K, int N_total) {
  // header (arrival counters, status word) + fp32 partial sums [slots][M][64] per tile.  With many tiles
  // a tile is shared by at most two blocks per k-part; with few tiles by at most one block per chunk
  // (+2 per k-part).  Tiles: 64-row tiles plus one ragged tile per kept block, blocks of >= 32 rows assumed
  // (the launch re-checks its exact need and returns UNIQL_ERR_WORKSPACE when this estimate is too small).
  if (M > 16) return (size_t)kWsHeader;
  DecodeCfg c;
  memset(&c, 0, sizeof(c));
  const int G = (K + kGroup - 1) / kGroup;
  if (!plan_split(&c, M, G, 2, false)) return (size_t)kWsHeader;
  const size_t chunks = (size_t)(G + CG - 1) / CG;
  const size_t tiles = (size_t)(N_total + RB - 1) / RB + (size_t)N_total / 32 + 2 * kMaxJobs;
  const size_t slots = tiles * 2 * c.n_kp + (size_t)c.n_rp * c.n_kp * (chunks + 2 * c.n_kp);
  // (+ the quantised activations of the streamed mode: 16 virtual rows of 128 bytes and 64 bytes per group, twice
  // that for more than eight rows)
  const size_t xs_group = M > 8 ? 2 * (16 * 128 + 64) : (16 * 128 + 64);
  return (size_t)kWsHeader + slots * (size_t)M * RB * 4 + (size_t)round_up(G, CG) * xs_group + 512;
}

int launch_decode(const Params& p, const LaunchCfg& cfg) {
  DecodeCfg c;
  memset(&c, 0, sizeof(c));
  const int G = p.K / kGroup;
  const int gran = copy_granule(G);
  int g_total = 0, v_first = 0;
  visited_range(p.imap, gran, &v_first, &g_total);
  const int MT = p.M <= 8 ? 1 : 2;
  // 128-bit staging: one leading family, everything 8-element aligned
  c.x_vec = decode_integer_path(p);
  if (count_tile_fams(p) > kMaxTF) return UNIQL_ERR_UNSUPPORTED;

  // integer path: fp16 activations staged with 128-bit loads (a leading input block); UNIQL_DECODE_I8=0: fp16 MMAs
  const bool i8 = c.x_vec && opt(kOptDecodeI8) != 0;
  // Streamed activations for rows too long to stage whole beside the ring (which would otherwise split the input
  // channels over several groups of blocks and hand every tile over); UNIQL_DECODE_XSTREAM=0/1 forces.  Where the
  // staged copy fits the quantising kernel in front costs more than the staging it saves (measured 3.5 us), and
  // inside a sequence of launches it only pays for itself from five rows on, where the staged copy would split
  // the input channels (Llama-3-8B gate|up + down at M = 5 / 6 / 7: 39.7 / 40.9 / 43.0 against 40.6 / 42.8 / 49.2 us;
  // at M <= 4, and wherever the staged copy fits whole, staging is faster).  Nine to sixteen rows are always
  // streamed: their staged copy never fits beside a ring of more than two positions (Llama-3-8B MLP at M = 16:
  // 55 us in one pass, 82 us as two launches of eight rows, 145 us with the input channels split over two groups
  // of blocks).
  size_t smem = 0;
  c.stage_bytes = STAGE_BYTES;
  {
    const int force = opt(kOptDecodeXstream);
    if (i8 && p.M > 8) {
      if (decode_streams_batch(p)) {
        smem = plan_stream(&c, p.M, g_total, gran);
        c.x_stream = smem != 0;
        if (!smem) c.stage_bytes = STAGE_BYTES;
      }
    } else if (i8 && force != 0) {
      DecodeCfg t = c;
      const size_t s0 = plan_split(&t, p.M, g_total, gran, true);
      if (force == 1 || !s0 || (t.n_kp > 1 && p.M >= 5)) {
        smem = plan_stream(&c, p.M, g_total, gran);
        c.x_stream = smem != 0;
        if (!smem) c.stage_bytes = STAGE_BYTES;
      }
    }
  }
  if (!c.x_stream) smem = plan_split(&c, p.M, g_total, gran, i8);
  if (!smem) return UNIQL_ERR_UNSUPPORTED;

  // ---- narrow tiles (32 rows x 16 groups) when the schedule they give is shorter: matrices with fewer
  //      64-row tiles than blocks then run without a hand-over between blocks (UNIQL_DECODE_NARROW=0/1 forces)
  bool narrow = false;
  {
    bool all_plain = true;
    long t64 = 0, t32 = 0;
    for (int j = 0; j < p.n_jobs; ++j) {
      const JobDev& jb = p.job[j];
      if (jb.rope.enabled) { all_plain = false; continue; }
      for (int k = 0; k < jb.omap.n_fam; ++k) {
        const Fam& a = jb.omap.fam[k];
        t64 += (long)((a.keep + RB - 1) / RB) * a.count;
        t32 += (long)((a.keep + RB / 2 - 1) / (RB / 2)) * a.count;
      }
    }
    if (all_plain && !c.x_stream) {
      const int Gk0 = g_total < c.gp ? g_total : c.gp;
      // (only where there are fewer wide tiles than blocks and the input channels are not split: measured,
      //  the smaller boxes of the narrow tiles cost more than a better balance of many tiles gains)
      narrow = c.n_kp == 1 && t64 < c.n_rp &&
               schedule_cost(t32, (Gk0 + 2 * CG - 1) / (2 * CG), c.n_rp) < schedule_cost(t64, (Gk0 + CG - 1) / CG, c.n_rp);
      const int force = opt(kOptDecodeNarrow);
      if (force == 0) narrow = false;
      if (force == 1) narrow = true;
    }
  }
  c.cgz = narrow ? 2 * CG : CG;

  // ---- tile families and their tensor maps
  const int x_extent = (v_first + g_total) * 64 < p.K / 2 ? (v_first + g_total) * 64 : p.K / 2;
  int tiles = 0, n_tf = 0;
  for (int j = 0; j < p.n_jobs; ++j) {
    const JobDev& jb = p.job[j];
    if (jb.rope.enabled) {
      const int half = jb.rope.head_keep / 2;
      TileFam& f = c.tf[n_tf];
      f.tile_begin = tiles; f.tpb = (half + RB / 2 - 1) / (RB / 2); f.keep = half; f.count = jb.rope.n_heads;
      f.job = j; f.start = 0; f.period = jb.rope.head_dim; f.out_base = 0; f.mode = kRope; f.job2 = j;
      const int rc = encode_family(&c.wmap[n_tf], jb.w, p.K, x_extent, half, 2 * jb.rope.n_heads,
                                   jb.rope.head_dim / 2, RB / 2);
      if (rc) return rc;
      tiles += f.tpb * f.count;
      ++n_tf;
    } else {
      const int rows = narrow ? RB / 2 : RB;
      for (int k = 0; k < jb.omap.n_fam; ++k) {
        const Fam& a = jb.omap.fam[k];
        TileFam& f = c.tf[n_tf];
        f.tile_begin = tiles; f.tpb = (a.keep + rows - 1) / rows; f.keep = a.keep; f.count = a.count;
        f.job = j; f.start = a.start; f.period = a.period; f.out_base = jb.omap.base[k];
        f.mode = narrow ? kNarrow : kPlain; f.job2 = j;
        const int rc = encode_family(&c.wmap[n_tf], jb.w + (size_t)a.start * (p.K / 2), p.K, x_extent, a.keep,
                                     a.count, a.count > 1 ? a.period : a.keep, rows);
        if (rc) return rc;
        tiles += f.tpb * f.count;
        ++n_tf;
      }
    }
  }
  c.n_tf = n_tf;
  c.tiles_total = tiles;
  for (int i = 0; i < n_tf; ++i) c.tf[i].by_tpb = fast_div((unsigned)c.tf[i].tpb, (unsigned long long)tiles);
  c.n_ph = 1;
  {
    Phase& P = c.ph[0];
    P.x = p.x; P.ldx = p.ldx; P.K = p.K;
    P.start = p.imap.fam[0].start; P.keep = p.imap.fam[0].keep;
    P.period = p.imap.fam[0].period; P.count = p.imap.fam[0].count;
    P.g_total = g_total; P.v_first = v_first;
    P.tile0 = 0; P.tiles = tiles;
    fill_split(c, &P);
    // Shared staging in clusters of two: integer path, activations staged whole by every block (no k-split, no
    // streaming, no block that stages only the chunks of a short run), blocks paired so that both have work or
    // neither has.  UNIQL_DECODE_XCLUSTER=0 turns it off.
    const bool all_stage_everything = P.base > 0 || P.R == 0 || (P.R * P.ck0) / P.bt0 >= P.ck0;
    const bool pairs_alike = P.base > 0 || (P.bt0 % 2) == 0;
    // Launching as clusters delays the start of the blocks (pairs of free SMs are needed, measured 1.5 - 2 us on the
    // small launches), so it is used where the staging is long: seven or eight rows and eight or more 16-byte units
    // per thread (smaller batches would alternate between two kernel functions within a layer, which costs more
    // than the staging saved).
    const int force_xc = opt(kOptDecodeXcluster);
    c.x_cluster = i8 && !c.x_stream && c.n_kp == 1 && (c.n_rp % 2) == 0 && p.M <= 8 && all_stage_everything &&
                  pairs_alike && force_xc != 0 && (force_xc == 1 || (p.M >= 7 && g_total * p.M >= 256));
  }
  if (tiles < 1 || tiles * EW > kCounterInts) return UNIQL_ERR_UNSUPPORTED;
  c.max_slots = slots_needed(tiles, c.g_total, c.gp, c.n_rp, c.cgz);
  size_t need = (size_t)kWsHeader + (size_t)tiles * c.max_slots * p.M * RB * 4;
  StreamWs sw;
  if (c.x_stream) need = stream_need(c, p.M, g_total, need, &sw);
  if (!cfg.workspace || cfg.ws_bytes < need) return UNIQL_ERR_WORKSPACE;
  unsigned char* ws = reinterpret_cast<unsigned char*>(cfg.workspace);
  c.counters = reinterpret_cast<int*>(ws);
  c.status = reinterpret_cast<int*>(ws + kStatusOff);
  c.partials = reinterpret_cast<float*>(ws + kWsHeader);
  c.grid_sync = reinterpret_cast<int*>(ws + kGridSyncOff);
  if (cfg.clear_header) {
    // every check has passed: only now is anything put on the stream.  What must start at zero: the counters of
    // this launch's tiles, the status word and the two counters of the barrier between phases.
    if (cudaMemsetAsync(ws, 0, (size_t)tiles * EW * sizeof(int), cfg.stream) != cudaSuccess ||
        cudaMemsetAsync(ws + kStatusOff, 0, 256, cfg.stream) != cudaSuccess) {
      cudaGetLastError();
      return UNIQL_ERR_CUDA;
    }
  }
  if (c.x_stream) {
    const int rc = stream_setup(c, c.ph[0], p.M, g_total, ws, sw, cfg.stream);
    if (rc != UNIQL_OK) return rc;
  }
  if (i8 && p.M > 4 && p.M <= 8) {
    // five to eight rows: one instance that can stream and share, whatever this launch does
    int rc = launch_t<1, false, 2, 1, true, true>(p, c, smem, cfg.stream);
    if (rc == UNIQL_ERR_UNSUPPORTED && c.x_cluster) {      // clusters cannot all be resident, or were refused
      c.x_cluster = 0;
      rc = launch_t<1, false, 2, 1, true, true>(p, c, smem, cfg.stream);
    }
    return rc;
  }
  if (c.x_stream && p.M > 8) return launch_t<2, false, 4, 1, true>(p, c, smem, cfg.stream);   // nine to sixteen rows, one launch
  if (c.x_stream) return launch_t<1, false, 1, 1, true>(p, c, smem, cfg.stream);      // (M <= 4: rows too long to stage)
  if (i8 && c.x_cluster) {                                                           // (M <= 4: forced only)
    const int rc = launch_t<1, false, 1, 1, false, true>(p, c, smem, cfg.stream);
    if (rc != UNIQL_ERR_UNSUPPORTED) return rc;
    c.x_cluster = 0;
  }
  if (i8) {
    if (p.M <= 4) return launch_t<1, false, 1, 1>(p, c, smem, cfg.stream);
    return launch_t<2, false, 4, 1>(p, c, smem, cfg.stream);
  }
  if (MT == 1)
    return p.M == 1 ? launch_t<1, true, 0, 1>(p, c, smem, cfg.stream) : launch_t<1, false, 0, 1>(p, c, smem, cfg.stream);
  return launch_t<2, false, 0, 1>(p, c, smem, cfg.stream);
}

// ---------------------------------------------------------------------------------------- SwiGLU MLP
int mlp_decode_supported(const MlpDecode& d) {
  if (d.M < 1 || d.M > 16) return 0;
  if (d.hidden < 2 * kGroup || d.inter < 2 * kGroup) return 0;
  if ((d.hidden % (2 * kGroup)) != 0 || (d.inter % (2 * kGroup)) != 0) return 0;
  if (d.k_int < 8 || d.k_int > d.inter || (d.k_int % 8) != 0) return 0;
  if ((d.ldx % 8) != 0 || (d.ldh % 8) != 0 || d.ldx < d.hidden || d.ldh < d.k_int || d.ldy < d.hidden) return 0;
  if ((((uintptr_t)d.x) | ((uintptr_t)d.h)) & 15) return 0;
  const int ga = copy_granule(d.hidden / kGroup), gb = copy_granule(d.inter / kGroup);
  if ((((uintptr_t)d.sg) | ((uintptr_t)d.zg) | ((uintptr_t)d.su) | ((uintptr_t)d.zu)) & (uintptr_t)(ga * 2 - 1)) return 0;
  if ((((uintptr_t)d.sd) | ((uintptr_t)d.zd)) & (uintptr_t)(gb * 2 - 1)) return 0;
  return 1;
}

size_t mlp_decode_workspace_bytes(int M, int hidden, int inter) {
  const size_t a = decode_workspace_bytes(M, hidden, 2 * inter);
  const size_t b = decode_workspace_bytes(M, inter, hidden);
  return a + b;      // the fused launch numbers the tiles of both products in one sequence
}

namespace {

// Phases [first, first + count) of the MLP (0: gate|up with the gated product as epilogue, 1: down) in one launch.
int launch_mlp_phases(const MlpDecode& d, int first, int count, const LaunchCfg& cfg) {
  Params p;
  memset(&p, 0, sizeof(p));
  p.x = first == 0 ? d.x : d.h;
  p.ldx = first == 0 ? d.ldx : d.ldh;
  p.dt = UNIQL_F16;
  p.M = d.M;
  p.K = first == 0 ? d.hidden : d.inter;
  p.k_in = first == 0 ? d.hidden : d.k_int;
  p.n_jobs = 3;
  JobDev& jg = p.job[0];
  JobDev& ju = p.job[1];
  JobDev& jd = p.job[2];
  jg.w = d.wg; jg.scales = d.sg; jg.zeros = d.zg; jg.y = d.h; jg.ldy = d.ldh; jg.N = d.inter; jg.k_out = d.k_int;
  ju.w = d.wu; ju.scales = d.su; ju.zeros = d.zu; ju.y = d.h; ju.ldy = d.ldh; ju.N = d.inter; ju.k_out = d.k_int;
  jd.w = d.wd; jd.scales = d.sd; jd.zeros = d.zd; jd.y = d.y; jd.ldy = d.ldy; jd.N = d.hidden; jd.k_out = d.hidden;

  DecodeCfg c;
  memset(&c, 0, sizeof(c));
  c.x_vec = 1;
  c.n_ph = count;
  c.stage_bytes = STAGE_BYTES;
  int g_max = 0, gran = 8;
  for (int ph = first; ph < first + count; ++ph) {
    const int g_total = ph == 0 ? d.hidden / kGroup : (d.k_int + kGroup - 1) / kGroup;
    if (g_total > g_max) g_max = g_total;
    const int gr = copy_granule((ph == 0 ? d.hidden : d.inter) / kGroup);
    if (gr < gran) gran = gr;
  }
  // (nine to sixteen rows: the gate|up launch on its own, activations streamed through the ring)
  const bool stream = count == 1 && first == 0 && d.M > 8 && opt(kOptDecodeSplitBatch) == 2 && opt(kOptDecodeXstream) != 0;
  size_t smem = stream ? plan_stream(&c, d.M, g_max, gran) : 0;
  c.x_stream = smem != 0;
  if (!smem) {
    c.stage_bytes = STAGE_BYTES;
    smem = plan_split(&c, d.M, g_max, gran, true);
  }
  if (!smem) return UNIQL_ERR_UNSUPPORTED;
  if (count > 1 && (c.n_kp != 1 || d.M > 8)) return UNIQL_ERR_UNSUPPORTED;
  // the down projection on its own: narrow tiles under the same rule as any plain launch
  bool narrow = false;
  if (first == 1 && count == 1) {
    const int Gk0 = g_max < c.gp ? g_max : c.gp;
    narrow = c.n_kp == 1 && (d.hidden + RB - 1) / RB < c.n_rp &&
             schedule_cost((d.hidden + RB / 2 - 1) / (RB / 2), (Gk0 + 2 * CG - 1) / (2 * CG), c.n_rp) <
                 schedule_cost((d.hidden + RB - 1) / RB, (Gk0 + CG - 1) / CG, c.n_rp);
    const int force = opt(kOptDecodeNarrow);
    if (force == 0) narrow = false;
    if (force == 1) narrow = true;
  }
  c.cgz = narrow ? 2 * CG : CG;

  int tiles = 0, n_tf = 0;
  for (int ph = first; ph < first + count; ++ph) {
    Phase& P = c.ph[ph - first];
    TileFam& f = c.tf[n_tf];
    f.tile_begin = tiles; f.count = 1; f.start = 0; f.out_base = 0;
    P.tile0 = tiles; P.v_first = 0;
    int rc;
    if (ph == 0) {
      P.x = d.x; P.ldx = d.ldx; P.K = d.hidden; P.start = 0; P.keep = d.hidden; P.g_total = d.hidden / kGroup;
      P.period = d.hidden; P.count = 1;
      f.mode = kSwiglu; f.job = 0; f.job2 = 1; f.keep = d.k_int; f.period = d.inter;
      f.tpb = (d.k_int + RB / 2 - 1) / (RB / 2);
      rc = encode_family(&c.wmap[n_tf], d.wg, d.hidden, d.hidden / 2, d.k_int, 1, d.k_int, RB / 2);
      if (!rc) rc = encode_family(&c.wmap_up, d.wu, d.hidden, d.hidden / 2, d.k_int, 1, d.k_int, RB / 2);
    } else {
      P.x = d.h; P.ldx = d.ldh; P.K = d.inter; P.start = 0; P.keep = d.k_int; P.period = d.inter; P.count = 1;
      P.g_total = (d.k_int + kGroup - 1) / kGroup;
      const int rows = narrow ? RB / 2 : RB;
      f.mode = narrow ? kNarrow : kPlain; f.job = 2; f.job2 = 2; f.keep = d.hidden; f.period = d.hidden;
      f.tpb = (d.hidden + rows - 1) / rows;
      const int x_extent = P.g_total * 64 < d.inter / 2 ? P.g_total * 64 : d.inter / 2;
      rc = encode_family(&c.wmap[n_tf], d.wd, d.inter, x_extent, d.hidden, 1, d.hidden, rows);
    }
    if (rc) return rc;
    P.tiles = f.tpb;
    tiles += f.tpb;
    ++n_tf;
  }
  c.n_tf = n_tf;
  c.tiles_total = tiles;
  for (int i = 0; i < n_tf; ++i) c.tf[i].by_tpb = fast_div((unsigned)c.tf[i].tpb, (unsigned long long)tiles);
  if (tiles < 1 || tiles * EW > kCounterInts) return UNIQL_ERR_UNSUPPORTED;
  c.max_slots = 0;
  for (int i = 0; i < count; ++i) fill_split(c, &c.ph[i]);
  for (int i = 0; i < count; ++i) {
    const int sl = slots_needed(c.ph[i].tiles, c.ph[i].g_total, c.gp, c.n_rp, c.cgz);
    if (sl > c.max_slots) c.max_slots = sl;
  }
  size_t need = (size_t)kWsHeader + (size_t)tiles * c.max_slots * d.M * RB * 4;
  StreamWs sw;
  if (c.x_stream) need = stream_need(c, d.M, c.ph[0].g_total, need, &sw);
  if (!cfg.workspace || cfg.ws_bytes < need) return UNIQL_ERR_WORKSPACE;
  unsigned char* ws = reinterpret_cast<unsigned char*>(cfg.workspace);
  c.counters = reinterpret_cast<int*>(ws);
  c.status = reinterpret_cast<int*>(ws + kStatusOff);
  c.partials = reinterpret_cast<float*>(ws + kWsHeader);
  c.grid_sync = reinterpret_cast<int*>(ws + kGridSyncOff);
  {
    const int shift = opt(kOptWaitShift);
    c.grid_wait_limit = shift > 0 ? (shift >= 21 ? 1 : kGridWaitLimit >> shift) : kGridWaitLimit;
  }
  if (c.x_stream) {
    const int rc = stream_setup(c, c.ph[0], d.M, c.ph[0].g_total, ws, sw, cfg.stream);
    if (rc != UNIQL_OK) return rc;
    return launch_t<2, false, 4, 1, true>(p, c, smem, cfg.stream);
  }
  if (count > 1) {
    if (d.M <= 4) return launch_t<1, false, 1, 2>(p, c, smem, cfg.stream);
    return launch_t<1, false, 2, 2>(p, c, smem, cfg.stream);
  }
  if (d.M <= 4) return launch_t<1, false, 1, 1>(p, c, smem, cfg.stream);
  if (d.M <= 8) {
    // shared staging under the rule of the plain launches (every block of the gate|up launch has whole tiles)
    const Phase& P = c.ph[0];
    const int force_xc = opt(kOptDecodeXcluster);
    c.x_cluster = c.n_kp == 1 && (c.n_rp % 2) == 0 && P.base > 0 && force_xc != 0 && d.M >= 7 && P.g_total * d.M >= 256;
    int rc = launch_t<1, false, 2, 1, true, true>(p, c, smem, cfg.stream);
    if (rc == UNIQL_ERR_UNSUPPORTED && c.x_cluster) {
      c.x_cluster = 0;
      rc = launch_t<1, false, 2, 1, true, true>(p, c, smem, cfg.stream);
    }
    return rc;
  }
  return launch_t<2, false, 4, 1>(p, c, smem, cfg.stream);
}

}  // namespace

int launch_mlp_decode(const MlpDecode& d, int fuse, const LaunchCfg& cfg) {
  if (!mlp_decode_supported(d)) return UNIQL_ERR_UNSUPPORTED;
  if (fuse) return launch_mlp_phases(d, 0, 2, cfg);
  const int rc = launch_mlp_phases(d, 0, 1, cfg);
  if (rc) return rc;
  // the down projection is an ordinary launch on h (leading k_int input channels, all hidden outputs): it takes
  // the narrow tiles, the streamed or shared staging of the plain path as they apply
  Params p;
  memset(&p, 0, sizeof(p));
  p.x = d.h; p.ldx = d.ldh; p.dt = UNIQL_F16; p.M = d.M; p.K = d.inter; p.k_in = d.k_int;
  p.imap.n_fam = 1; p.imap.total = d.k_int; p.imap.fam[0] = Fam{0, d.k_int, d.k_int, 1}; p.imap.base[0] = 0;
  p.n_jobs = 1;
  JobDev& jd = p.job[0];
  jd.w = d.wd; jd.scales = d.sd; jd.zeros = d.zd; jd.y = d.y; jd.ldy = d.ldy; jd.N = d.hidden; jd.k_out = d.hidden;
  jd.omap.n_fam = 1; jd.omap.total = d.hidden; jd.omap.fam[0] = Fam{0, d.hidden, d.hidden, 1}; jd.omap.base[0] = 0;
  return launch_decode(p, cfg);
}

int decode_status_offset() { return kStatusOff; }
size_t decode_workspace_header_bytes() { return (size_t)kWsHeader; }

}  // namespace uniql
