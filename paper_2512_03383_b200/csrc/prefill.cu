// Prefill kernel (every batch the decode kernel does not take: more than 16 rows, bf16) of the pruned 4-bit
// linear layer, sm_100a: a dense contraction on
// the fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// Orientation.  The packed weights are four times smaller than the activations, so the weight side
// takes the MMA's M dimension (128 retained weight rows per tile, de-quantised once per tile and
// k-block) and the tokens its N dimension (up to 256 per tile): D[row][token] += W[row][k] x[token][k].
//
// Roles inside a block (one persistent block per SM, tiles taken round-robin):
//   warp 0       TMA producer: boxes [64 k x BN tokens] of activations into a ring of four (128-byte swizzle);
//                one box per k-block, or two where a tile takes both accumulators (512 tokens)
//   warp 1       allocates tensor memory; one lane issues the MMAs of a k-block (4 x K=16 per box) and commits
//                them to the box's and the weight stage's "empty" barriers and, at the end of a tile, to
//                "accumulator full"
//   warps 4..7   epilogue: tcgen05.ld the fp32 accumulators (warp w owns TMEM lanes 32(w-4).., a lane
//                is a tile row and holds 32 tokens of it per pass), bias, rotary embedding on the
//                retained pair (Section 3.2; the pair's two rows are neighbouring lanes and swap
//                values by shuffle), one rounding, stores of 32 consecutive outputs of a token per
//                warp; two accumulator buffers of 256 columns let the epilogue of tile i overlap
//                the MMAs of tile i+1 (tiles of 512 tokens use both and hand them back one by one);
//                the epilogue of a block's last tile is shared with the de-quantiser warps, idle by then
//   warps 8..23  de-quantisers: the twelve of them whose scheduler does not host the MMA warp (warp % 4 != 1), two
//                teams of six warps on alternate stages; a thread converts 32 codes of a weight row per item --
//                nibbles to fp16 by magic number, (q-8) exact, then one fp16 FMA (q-8)*s + fp16(s*(8-z))
//                -- and writes them into the A-operand stage in the
//                canonical K-major 128-byte-swizzled layout; the packed codes of the next k-block
//                are already in registers.  All sixteen share the epilogue of the block's last segment.
// Work split (chosen by the launcher from a cost model): whole tiles round-robin; tiles left over after the whole
// rounds split along K over all blocks (stream-K: parts handed over through slots in the workspace, or added into
// one sum per tile) or, for tiles of two boxes, run as half tiles on twice the blocks; launches with few tiles as
// clusters of two blocks per tile, the second block's sums written into the first one's idle rings.
// Launched with programmatic stream serialization: what a block does before griddepcontrol.wait (barriers, tensor
// memory, the first weight stages) touches nothing a preceding kernel may still read or write.
// On-device pruning (Section 3.4) is index arithmetic: tile rows are compact output channels mapped to
// stored rows per thread; the input side is the leading k_in channels (the TMA tensor ends at k_in, so
// the tail of the last k-block is zero activations).
// bf16 activations: bf16 weights would carry 2^-9 relative rounding error each, which alone spends the
// 2e-3 error budget; instead the de-quantisers convert the activation tile to fp16 in place (exact in
// fp16's range, saturating beyond) and both operands are fp16.
//
// Every mbarrier wait is bounded; on expiry the block raises a flag, every role leaves its loop, the
// status word of the workspace is set, tensor memory is released and the block returns.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace uniql {
namespace {

constexpr int BMW = 128;            // weight rows per tile (MMA M)
constexpr int BK = 64;              // k per stage: 128 bytes of fp16 / bf16, one swizzle row
constexpr int MAXBN = 256;          // tokens per tile (MMA N), at most
constexpr int PSTAGES = 4;                   // ring of de-quantised weight stages (one k-block each)
constexpr int BSLOTS = 4;                    // ring of activation boxes (one k-block of MAXBN tokens each)
constexpr int A_BYTES = BMW * BK * 2;        // 16 KB
constexpr int B_BYTES = MAXBN * BK * 2;      // 32 KB
constexpr int RING_BYTES = PSTAGES * A_BYTES + BSLOTS * B_BYTES;
constexpr int B_RING = PSTAGES * A_BYTES;    // the activation boxes follow the weight stages
constexpr int EPI_TOK = 32;                  // tokens per epilogue pass
constexpr int NWARPS = 24;
constexpr int PTH = NWARPS * 32;
constexpr int DQ_WARP0 = 8, DQ_WARPS = 8;      // warps 8 .. 8 + 2 * DQ_WARPS - 1: the de-quantisers and epilogue helpers
constexpr int DQ_TEAM_WARPS = 6;               // twelve of them convert: two teams of six warps on alternate stages
constexpr int EPI_WARP0 = 4;
constexpr int kPWait = 1 << 20;
constexpr int kMaxPJobs = kMaxJobs;

struct PrefillCfg {
  CUtensorMap xmap;          // activations: (k, token), box 64 x BN, 128-byte swizzle
  int bn;                    // tokens per MMA and activation box: 64, 128 or 256
  int nh;                    // boxes per tile: 2 when the tile takes both accumulators (512 tokens), else 1
  int n_ttiles;              // token tiles
  int wtile_begin[kMaxPJobs + 1];   // first weight tile of each job
  int n_tiles;               // weight tiles (all jobs) x token tiles
  int n_kb;                  // visited k-blocks of 64: kept blocks of every head, head after head
  int km_start, km_period;   // input map in k-blocks: first stored block of head 0, stored blocks per head
  int km_kbh, km_keep;       // kept k-blocks per head (the last may be partly kept), kept channels per head
  uint32_t idesc;
  int streamk;               // 1: contiguous ranges of (tile, k-block) units per block; 0: whole tiles round-robin
  int helpers;               // 1: the de-quantiser warps share the epilogue of the block's last tile
  int sk_atomic;             // stream-K hand-over: 1 = parts added into one sum per tile (reductions in L2), 0 = a slot per part
  int pair_split;            // clusters of two blocks on one tile, half of the contraction each; the second block's
                             // fp32 sums go into the first one's shared memory (the rings, idle by then)
  int halves;                // tiles on both accumulators: the tiles left over after the whole rounds run as half tiles
                             // (one box of 256 tokens each, on twice as many blocks), every block's last segment
  int* status;
  int* counters;             // stream-K: arrivals per tile
  float* partials;           // stream-K: one slot [tokens / 32][128 rows][32 tokens] fp32 per (left-over tile, block) piece
};

// Work of a block as a sequence of segments (tile, k-blocks [kb0, kb1)): whole tiles t = b, b + grid, ...
// With stream-K only for as many rounds as fill every block; the k-blocks of the tiles left over are
// cut into equal contiguous ranges, one per block, so that every SM stays busy however few tiles remain.
// A block runs its range of the split tiles FIRST: handing over the partial tile and finishing the split
// tiles then overlap the main loop of the whole tiles that follow instead of standing at the kernel's end.  Blocks stay in step along k (few distinct k offsets are alive at a time, which keeps the
// activation slices in L2).  Every block adds its fp32 partial tile to the tile's accumulation buffer in the
// workspace (reductions done in L2); the last of the tile's blocks to arrive reads the sum
// and finishes the tile.  With more than two blocks on a tile the order of the additions, and so the last
// bit of the fp32 sum, depends on the order of arrival.
// Visited k-block v of the input map -> stored k-block, first compact activation column, kept channels in it.
// One family {start, period, keep, count}: head h keeps channels [0, keep) of its period; a leading block is
// the case count = 1.  The activation box of a partly kept block also covers the first columns of the next
// head: the de-quantisers write zeros for the pruned channels of the block, so those columns do not count.
// Walked without a division per k-block (a division by the kept blocks per head cost the per-head launches 8 us
// of 52): (head, kept block within the head) of a visited k-block, stepped.
struct KWalk {
  int h, r;
  __device__ inline void start(const PrefillCfg& c, int v) { h = v / c.km_kbh; r = v - h * c.km_kbh; }
  __device__ inline void step(const PrefillCfg& c, int n) { r += n; while (r >= c.km_kbh) { r -= c.km_kbh; ++h; } }
  __device__ inline int stored(const PrefillCfg& c) const { return c.km_start + h * c.km_period + r; }
  __device__ inline int xcol(const PrefillCfg& c) const { return h * c.km_keep + r * BK; }
  __device__ inline int valid(const PrefillCfg& c) const { return min(BK, c.km_keep - r * BK); }
};

// half: -1 the whole tile; 0 / 1: only the first / second box of a tile of two boxes (into accumulator 0 / 1)
struct Seg { int tile, kb0, kb1, half; };
struct SegIter {
  long u, ue;
  int t, t_end, n_kb, step, tail_tile0, half_tile, half, ps_tile, ps_kb0, ps_kb1;
  __device__ inline void init(const PrefillCfg& c, int b, int grid) {
    n_kb = c.n_kb; step = grid; t = b;
    half_tile = -1; half = 0;
    ps_tile = -1;
    if (c.pair_split) {
      // block 2t takes the first k-blocks of tile t and finishes it, block 2t + 1 the rest (the smaller half)
      t_end = 0; tail_tile0 = 0; u = ue = 0; t = 1;
      ps_tile = b >> 1;
      const int mid = n_kb - n_kb / 2;
      ps_kb0 = (b & 1) ? mid : 0;
      ps_kb1 = (b & 1) ? n_kb : mid;
      return;
    }
    if (c.halves) {
      // whole rounds of whole tiles, then tile (rounds * grid + b / 2) as two halves on blocks b and b + 1
      const int full = (c.n_tiles / grid) * grid;
      t_end = full; tail_tile0 = full; u = ue = 0;
      if (full + b / 2 < c.n_tiles) { half_tile = full + b / 2; half = b & 1; }
      return;
    }
    const int base = c.streamk ? c.n_tiles / grid : (c.n_tiles + grid - 1) / grid;
    t_end = c.streamk ? base * grid : c.n_tiles;
    tail_tile0 = base * grid;
    u = ue = 0;
    if (c.streamk) {
      const long Ut = (long)(c.n_tiles - tail_tile0) * c.n_kb;
      const long Bt = grid < Ut ? grid : Ut;
      if (b < Bt) { u = Ut * b / Bt; ue = Ut * (b + 1) / Bt; }
    }
  }
  __device__ inline bool next(Seg& sg) {
    if (u < ue) {
      const int tt = (int)(u / n_kb);
      sg.tile = tail_tile0 + tt;
      sg.kb0 = (int)(u - (long)tt * n_kb);
      const long len = (n_kb - sg.kb0) < (ue - u) ? (n_kb - sg.kb0) : (ue - u);
      sg.kb1 = sg.kb0 + (int)len;
      sg.half = -1;
      u += len;
      return true;
    }
    if (t < t_end) {
      sg.tile = t; sg.kb0 = 0; sg.kb1 = n_kb; sg.half = -1;
      t += step;
      return true;
    }
    if (ps_tile >= 0) {
      sg.tile = ps_tile; sg.kb0 = ps_kb0; sg.kb1 = ps_kb1; sg.half = -1;
      ps_tile = -1;
      return true;
    }
    if (half_tile >= 0) {
      sg.tile = half_tile; sg.kb0 = 0; sg.kb1 = n_kb; sg.half = half;
      half_tile = -1;
      return true;
    }
    return false;
  }
};
// block whose range [U*b/B, U*(b+1)/B) of the left-over units holds unit u (exact in fp64 for these magnitudes)
__device__ inline int sk_owner(long u, long B, long U) {
  return (int)floor(((double)(u + 1) * (double)B - 1.0) / (double)U);
}

// ---------------------------------------------------------------------------------------- PTX
__device__ inline void pmbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ inline void pmbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ inline void pmbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ inline bool pmbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// `relaxed`: sleep between polls (roles that run several stages ahead and must not steal issue slots)
__device__ inline bool pmbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, bool relaxed = false) {
  for (int i = 0; i < kPWait; ++i) {
    if (pmbar_try(bar, parity)) return true;
    if (relaxed) __nanosleep(200);
    if ((i & 63) == 63 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// ---- clusters of two (a tile's contraction split over a pair of blocks)
__device__ inline uint32_t pcluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of `addr` (shared memory of this block) in block `rank` of the cluster
__device__ inline uint32_t ppeer_addr(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// generic address of `ptr` (shared memory of this block) in block `rank` of the cluster
__device__ inline float* ppeer_generic(void* ptr, uint32_t rank) {
  unsigned long long r;
  asm volatile("mapa.u64 %0, %1, %2;" : "=l"(r) : "l"(reinterpret_cast<unsigned long long>(ptr)), "r"(rank));
  return reinterpret_cast<float*>(r);
}
template <int STRIDE, int K = 0>
__device__ inline void pld_add_f32x16(uint32_t base, const uint32_t (&v)[16], float (&val)[16]) {
  if constexpr (K < 16) {
    float o;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(o) : "r"(base), "n"(K * STRIDE) : "memory");
    val[K] = __uint_as_float(v[K]) + o;
    pld_add_f32x16<STRIDE, K + 1>(base, v, val);
  }
}
__device__ inline void pmbar_arrive_peer(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ inline bool pmbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < kPWait; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    __nanosleep(100);
    if ((i & 63) == 63 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ inline void tma_box2(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ inline void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ inline void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ inline void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem desc] * B[smem desc]; accumulate == 0 overwrites D
__device__ inline void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on `bar` when all MMAs issued so far by this thread have completed
__device__ inline void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ inline void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ inline void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ inline void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ inline void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 fp16/bf16), 128-byte
// swizzle: 8-row groups 1024 bytes apart (stride byte offset), leading byte offset unused (1),
// descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ inline uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ inline uint32_t pand_or(uint32_t a, uint32_t mask, uint32_t magic) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(magic));
  return d;
}

// ---------------------------------------------------------------------------------------- tile rows
// Row r (0..127) of local weight tile `tl` of a job: stored weight row, or -1 when the row is empty.
// Rope jobs: rows 2i and 2i + 1 are the two members of rotation pair i (first-half member, then its partner),
// so that the two sit in neighbouring lanes of the epilogue warp that rotates them.  SwiGLU pairs (pair == 1)
// likewise: rows 2i and 2i + 1 are retained row i of the gate matrix and of the up matrix.
struct RowInfo { int stored; int out_col; int pair_c; int head; };
__device__ inline RowInfo tile_row(const JobDev& jb, int tl, int r) {
  RowInfo o;
  o.stored = -1; o.out_col = -1; o.pair_c = 0; o.head = 0;
  if (jb.rope.enabled) {
    const int half = jb.rope.head_keep >> 1;
    const int P = tl * (BMW / 2) + (r >> 1);
    if (P >= jb.rope.n_heads * half) return o;
    const int h = P / half, cc = P - h * half, hi = r & 1;
    o.stored = h * jb.rope.head_dim + hi * (jb.rope.head_dim >> 1) + cc;
    o.out_col = h * jb.rope.head_keep + hi * half + cc;
    o.pair_c = cc; o.head = h;
  } else if (jb.pair == 1) {
    const int j = tl * (BMW / 2) + (r >> 1);
    if (j >= jb.k_out) return o;
    o.stored = (jb.omap.n_fam == 1 && jb.omap.fam[0].count == 1) ? jb.omap.fam[0].start + j
                                                                  : map_compact_to_stored(jb.omap, j);
    o.out_col = j;
    o.pair_c = r & 1;          // 0: row of the gate matrix, 1: row of the up matrix
  } else {
    const int j = tl * BMW + r;
    if (j >= jb.k_out) return o;
    o.stored = (jb.omap.n_fam == 1 && jb.omap.fam[0].count == 1) ? jb.omap.fam[0].start + j
                                                                  : map_compact_to_stored(jb.omap, j);
    o.out_col = j;
  }
  return o;
}

// Two bf16 values of a word as two fp16 values (exact for magnitudes in fp16's normal range, which
// holds LLM activations; larger magnitudes saturate at +-65504 instead of becoming infinite).
__device__ inline uint32_t bf16x2_to_f16x2(uint32_t w) {
  uint32_t d;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(__uint_as_float(w & 0xffff0000u)), "f"(__uint_as_float(w << 16)));
  return d;
}

// Eight codes of one 32-bit word, in input-channel order, as eight fp16 values packed in a uint4:
// byte b -> (1024 + c_even, 64 + c_odd) as an fp16 pair (one PRMT, one LOP3), minus (1032, 72) = the
// exact (c-8) pair, then one fp16 FMA per pair: (c-8)*s + cz with cz = fp16(s*(8-z)).  s is the stored
// fp16 scale itself, (c-8)*s + cz is rounded once; the only other error is the rounding of cz (2^-12
// of at most 8 s, shared by the 128 weights of a group).
__device__ inline uint4 dequant_word(uint32_t w, __half2 s2, __half2 cz2) {
  uint32_t o[4];
  const __half2 off = __halves2half2(__ushort_as_half(0x6408), __ushort_as_half(0x5480));
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const uint32_t t = __byte_perm(w, 0u, 0x4040u + 0x0101u * b);
    const uint32_t v = pand_or(t, 0x00f0000fu, 0x54006400u);
    const __half2 r = __hfma2(__hsub2(*reinterpret_cast<const __half2*>(&v), off), s2, cz2);
    o[b] = *reinterpret_cast<const uint32_t*>(&r);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// bf16 activations -> fp16 copy in the workspace, once per call (every weight tile re-reads the tile of
// activations, so converting there would repeat the work once per 128 weight rows).
__global__ void x_to_f16_kernel(const __nv_bfloat16* __restrict__ x, int ldx, int M, int k_in, __half* __restrict__ o, int ldo) {
  // (programmatic dependent launch: the tensor-core kernel behind this one may set itself up meanwhile; this one
  //  waits for its own predecessor before it reads x or overwrites the copy that predecessor may still read)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int units = ldo / 8;                         // 16-byte units per output row (ldo is a multiple of 8)
  const long total = (long)M * units;
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int m = (int)(i / units), u = (int)(i - (long)m * units);
    const __nv_bfloat16* src = x + (size_t)m * ldx + u * 8;
    uint32_t w[4];
    if (u * 8 + 8 <= k_in && ((ldx & 7) == 0) && ((((uintptr_t)x) & 15) == 0)) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
      w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int k0 = u * 8 + 2 * e;
        const uint32_t lo = k0 < k_in ? __bfloat16_as_ushort(src[2 * e]) : 0u;
        const uint32_t hi = k0 + 1 < k_in ? __bfloat16_as_ushort(src[2 * e + 1]) : 0u;
        w[e] = lo | (hi << 16);
      }
    }
    uint4 r;
    r.x = bf16x2_to_f16x2(w[0]); r.y = bf16x2_to_f16x2(w[1]); r.z = bf16x2_to_f16x2(w[2]); r.w = bf16x2_to_f16x2(w[3]);
    *reinterpret_cast<uint4*>(o + (size_t)m * ldo + u * 8) = r;
  }
}

// T: activation / output type.  CONV: the activation tiles arrive as bf16 and are converted to fp16 in
// shared memory by the de-quantisers (used when the workspace cannot hold a converted copy).
// HEADS: the input map is a family of per-head blocks (else a leading block).
template <typename T, bool CONV, bool HEADS>
__global__ void __launch_bounds__(PTH, 1) prefill_kernel(const __grid_constant__ Params p,
                                                         const __grid_constant__ PrefillCfg c) {
  extern __shared__ unsigned char psmem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Programmatic dependent launch: the next kernel of the stream may be set up while this one runs (its blocks
  // become resident as ours leave).  What a block does before its own `griddepcontrol.wait` touches nothing a
  // predecessor may still write or read: barriers, tensor memory, and the weights, which no kernel writes (the
  // de-quantisers fill the ring ahead); activations, positions, outputs and workspace come after the wait.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t raw = (uint32_t)__cvta_generic_to_shared(psmem_raw);
  const uint32_t sbase = (raw + 1023u) & ~1023u;           // swizzled tiles need 1024-byte alignment
  unsigned char* smem = psmem_raw + (sbase - raw);
  const uint32_t bars = sbase + RING_BYTES;
  const uint32_t full_a = bars, empty_a = bars + 8 * PSTAGES;
  const uint32_t full_b = bars + 16 * PSTAGES, empty_b = full_b + 8 * BSLOTS;
  const uint32_t acc_full = full_b + 16 * BSLOTS, acc_empty = acc_full + 16, epi_bar = acc_full + 32;
  const uint32_t help_bar = acc_full + 40;         // the epilogue warps and the de-quantiser warps that help them
  const uint32_t last_full = acc_full + 48;        // the MMAs of the block's last segment are complete (one phase only)
  const uint32_t px_ready = acc_full + 56;         // pair split, second block: the first block's rings are idle
  const uint32_t px_done = acc_full + 64;          // pair split, first block: the second block's sums have arrived
  unsigned char* misc = smem + RING_BYTES + 16 * PSTAGES + 16 * BSLOTS + 72;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);

  if (tid == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      pmbar_init(full_a + 8 * s, DQ_TEAM_WARPS);
      pmbar_init(empty_a + 8 * s, 1);
    }
    for (int s = 0; s < BSLOTS; ++s) {
      pmbar_init(full_b + 8 * s, 1);
      pmbar_init(empty_b + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) { pmbar_init(acc_full + 8 * b, 1); pmbar_init(acc_empty + 8 * b, 4); }
    pmbar_init(epi_bar, 4);
    pmbar_init(help_bar, 4 + 2 * DQ_WARPS);
    pmbar_init(last_full, 1);
    pmbar_init(px_ready, 1);
    pmbar_init(px_done, c.helpers ? 4 + 2 * DQ_WARPS : 4);       // one arrival per warp that sends
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                      // the whole tensor memory of the SM: two accumulators of 256 columns
    tmem_alloc((uint32_t)__cvta_generic_to_shared(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t crank = c.pair_split ? pcluster_rank() : 0u;
  if (c.pair_split) {                   // the other block's barriers exist before anything is sent to it
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }

  auto job_of_wt = [&](int wt) { int j = 0; while (j + 1 < p.n_jobs && wt >= c.wtile_begin[j + 1]) ++j; return j; };
  bool failed = false;

  // ---- the epilogue of one segment, for the warp that calls it: accumulator -> bias, rotary embedding or gated
  //      product, rounding, store.  A warp reaches the tensor-memory lanes 32 (warp % 4) .. + 31 (a lane is a tile
  //      row); it takes the chunks ch0, ch0 + chs, ... of 32 tokens.  chs == 1: the epilogue warp on its own (it
  //      also hands the accumulators back and runs the hand-over of a tile split along K).
  const int q = warp & 3;                          // TMEM lanes 32q .. 32q+31
  const int etid = 32 * q + lane;                  // tile row handled in the store phase
  uint32_t epar = 0;
  auto epi_sync = [&]() -> bool {
    __syncwarp();
    if (lane == 0) pmbar_arrive(epi_bar);
    const bool ok = pmbar_wait(epi_bar, epar, abort_flag);
    epar ^= 1;
    return ok;
  };
  volatile int* last_flag = reinterpret_cast<volatile int*>(misc + 8);
  uint32_t hpar = 0;
  auto help_sync = [&]() -> bool {
    __syncwarp();
    if (lane == 0) pmbar_arrive(help_bar);
    const bool ok = pmbar_wait(help_bar, hpar, abort_flag);
    hpar ^= 1;
    return ok;
  };
  auto epilogue_segment = [&](const Seg& sg, int tcount, int ch0, int chs, bool acc_known_full) {
      const int acc0 = c.nh == 2 ? 0 : (tcount & 1);     // as in the MMA warp
      const int au = c.nh == 2 ? tcount : (tcount >> 1);
      const int ntok = c.bn * c.nh;                      // tokens of the tile
      const int h_lo = sg.half < 0 ? 0 : sg.half, h_hi = sg.half < 0 ? c.nh : sg.half + 1;   // boxes of this segment
      const int t = sg.tile;
      const int wt = t / c.n_ttiles, tt = t - wt * c.n_ttiles;
      const int jn = job_of_wt(wt);
      const JobDev& jb = p.job[jn];
      const int tl = wt - c.wtile_begin[jn];
      T* y = reinterpret_cast<T*>(jb.y);
      const T* bias = reinterpret_cast<const T*>(jb.bias);
      const bool rope = jb.rope.enabled != 0;
      // this thread owns tile row etid (= its TMEM lane); a rope pair sits in lanes 2i, 2i + 1
      const RowInfo ri = tile_row(jb, tl, etid);
      float b_own = 0.f;
      unsigned long long turn = 0;
      const bool swiglu = jb.pair == 1;
      if (ri.stored >= 0) {
        const T* bias_own = (swiglu && (etid & 1)) ? reinterpret_cast<const T*>(p.job[jn + 1].bias) : bias;
        if (bias_own) b_own = DT<T>::to_f(bias_own[ri.stored]);
        if (rope) {
          const int half = jb.rope.head_keep >> 1;
          int pidx = p.idx[(ri.head / jb.rope.rep) * half + ri.pair_c];
          pidx = min(max(pidx, 0), (jb.rope.head_dim >> 1) - 1);
          turn = p.rope_turn[pidx];
        }
      }
      // bias, rotary embedding, rounding and store of 32 tokens of this row (all lanes of the warp call it)
      auto store_chunk = [&](int tok0, const auto& val) {
        constexpr int NV = (int)(sizeof(val) / sizeof(float));
        const int m0 = tt * ntok + tok0;
        if (rope) {
          // the even lane of a pair rotates the even tokens, the odd lane the odd ones: one exchange hands
          // each the other member's value of its token, and it stores both rotated members
          const bool second = (lane & 1) != 0;
          const int half = jb.rope.head_keep >> 1;
          const float b_other = __shfl_xor_sync(0xffffffffu, b_own, 1);
          const float b_lo = second ? b_other : b_own, b_hi = second ? b_own : b_other;
          const bool live = ri.stored >= 0;
          const int left = p.M - m0, odd = second ? 1 : 0;
          T* yp = y + (live ? ri.out_col - (second ? half : 0) : 0) + (size_t)(m0 + odd) * jb.ldy;   // this lane's first token
          const size_t step = 2 * (size_t)jb.ldy;
          const int32_t* pp = p.pos + m0 + odd;
          if (left >= NV) {                       // a whole chunk of tokens: no test per token
#pragma unroll
            for (int k = 0; k < NV; k += 2) {
              const float got = __shfl_xor_sync(0xffffffffu, second ? val[k] : val[k + 1], 1);
              const float lo = (second ? got : val[k]) + b_lo, hi = (second ? val[k + 1] : got) + b_hi;
              float cs, sn;
              rope_cos_sin(__ldg(pp + k), turn, cs, sn);
              if (live) {
                yp[0] = DT<T>::from_f(fmaf(-hi, sn, lo * cs));
                yp[half] = DT<T>::from_f(fmaf(lo, sn, hi * cs));
              }
              yp += step;
            }
          } else {
#pragma unroll
            for (int k = 0; k < NV; k += 2) {
              if (k >= left) break;
              const float got = __shfl_xor_sync(0xffffffffu, second ? val[k] : val[k + 1], 1);
              const float lo = (second ? got : val[k]) + b_lo, hi = (second ? val[k + 1] : got) + b_hi;
              if (live && k + odd < left) {
                float cs, sn;
                rope_cos_sin(__ldg(pp + k), turn, cs, sn);
                yp[0] = DT<T>::from_f(fmaf(-hi, sn, lo * cs));
                yp[half] = DT<T>::from_f(fmaf(lo, sn, hi * cs));
              }
              yp += step;
            }
          }
        } else if (swiglu) {
          // as for a rotation pair: the even lane (gate row) takes the even tokens, the odd lane (up row) the odd
          // ones, one exchange gives each the other matrix's sum of its token; h = silu(g) * u, one rounding
          // (the approximate division: two instructions instead of ten in warps that share the issue slots
          //  with the de-quantisers; exp(-g) beyond fp32 gives a quotient of zero, the limit of silu)
          const bool second = (lane & 1) != 0;
          const float b_other = __shfl_xor_sync(0xffffffffu, b_own, 1);
          const float b_g = second ? b_other : b_own, b_u = second ? b_own : b_other;
          const bool live = ri.stored >= 0;
          const int left = p.M - m0, odd = second ? 1 : 0;
          T* yp = y + (live ? ri.out_col : 0) + (size_t)(m0 + odd) * jb.ldy;          // this lane's first token
          const size_t step = 2 * (size_t)jb.ldy;
          if (left >= NV) {                       // a whole chunk of tokens: no test per token
#pragma unroll
            for (int k = 0; k < NV; k += 2) {
              const float got = __shfl_xor_sync(0xffffffffu, second ? val[k] : val[k + 1], 1);
              const float g = (second ? got : val[k]) + b_g, u = (second ? val[k + 1] : got) + b_u;
              if (live) *yp = DT<T>::from_f(__fdividef(g, 1.f + __expf(-g)) * u);
              yp += step;
            }
          } else {
#pragma unroll
            for (int k = 0; k < NV; k += 2) {
              if (k >= left) break;
              const float got = __shfl_xor_sync(0xffffffffu, second ? val[k] : val[k + 1], 1);
              const float g = (second ? got : val[k]) + b_g, u = (second ? val[k + 1] : got) + b_u;
              if (live && k + odd < left) *yp = DT<T>::from_f(__fdividef(g, 1.f + __expf(-g)) * u);
              yp += step;
            }
          }
        } else {
          if (ri.stored < 0) return;
          T* yr = y + ri.out_col + (size_t)m0 * jb.ldy;
          const int left = p.M - m0;
          if (left >= NV) {                       // a whole chunk of tokens: no test per token
#pragma unroll
            for (int k = 0; k < NV; ++k) { *yr = DT<T>::from_f(val[k] + b_own); yr += jb.ldy; }
          } else {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
              if (k >= left) break;
              *yr = DT<T>::from_f(val[k] + b_own);
              yr += jb.ldy;
            }
          }
        }
      };
      for (int h = h_lo; h < h_hi && !failed && !acc_known_full; ++h)
        if (!pmbar_wait(acc_full + 8 * (acc0 + h), au & 1, abort_flag)) failed = true;
      if (failed) return;
      tc_fence_after();
      // (the two accumulators are neighbours in tensor memory: a tile of two boxes is 512 consecutive columns)
      const uint32_t t_acc = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc0 * MAXBN);
      const int row = 32 * q + lane;
      // this warp is done with the accumulator that holds token chunk `ch` once that chunk was its last
      auto release_after = [&](int ch) {
        if (((ch + 1) * EPI_TOK) % c.bn != 0) return;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) pmbar_arrive(acc_empty + 8 * (acc0 + (ch * EPI_TOK) / c.bn));
      };
      if (sg.kb0 == 0 && sg.kb1 == c.n_kb) {
        // ---- the whole contraction of this tile ran here (this warp takes every chs-th chunk of 32 tokens;
        //      of a half tile only the chunks of its box)
        const int cpb = c.bn / EPI_TOK;
        for (int ch = h_lo * cpb + ch0; ch < h_hi * cpb; ch += chs) {
          uint32_t v[32];
          tmem_ld32(t_acc + (uint32_t)(ch * EPI_TOK), v);
          tmem_ld_wait();
          if (chs == 1) release_after(ch);               // (the values are in registers)
          float val[32];
#pragma unroll
          for (int k = 0; k < 32; ++k) val[k] = __uint_as_float(v[k]);
          store_chunk(ch * EPI_TOK, val);
        }
      } else {
        // ---- a part of the contraction (stream-K): the fp32 partial tile goes to a slot of its own in the
        //      workspace, [token][row] (a warp writes and later reads 32 consecutive rows of a token: whole
        //      128-byte lines); the last of the tile's blocks to arrive adds the slots of all of them in block
        //      order (the same sum whatever the order of arrival) and finishes the tile.
        //      The pieces (tile, block) of the cut unit line are numbered lt + block: both grow along the line and
        //      one of them grows from each piece to the next, so no two pieces share a number.
        //      chs > 1: the block's last segment, shared with the de-quantiser warps (twenty warps write, meet at a
        //      barrier of their own, and -- in the last block to arrive -- read back and finish).
        //      Where a few split tiles in front of whole tiles have many parts each, reading all the slots back
        //      would take the four epilogue warps longer than the tiles behind can hide: such launches add the parts
        //      into ONE sum per tile instead (reductions done in L2, zero at launch; the last bit of a sum then
        //      depends on the order of arrival when more than two blocks share a tile).
        const bool pair_send = c.pair_split && crank != 0;
        if (c.pair_split && !pair_send) {
          // ---- the two blocks of a cluster each ran half of the contraction.  The second block waits until the
          //      first one's MMAs are complete (its rings are idle then), writes its fp32 sums into them ([token][row]:
          //      a warp stores 32 consecutive rows of a token) and arrives, one arrival per warp, at the first block's
          //      barrier; the first block adds them to its own sums (always own + other: the same bits every run)
          //      and finishes the tile.  No traffic through L2, no counter, nothing to clear.
          {
            if (!pmbar_wait_cluster(px_done, 0, abort_flag)) { failed = true; return; }
            // (16 tokens at a time, as the read-back of the slots: what the registers of a thread hold)
            for (int tk = 16 * ch0; tk < ntok; tk += 16 * chs) {
              uint32_t v[16];
              tmem_ld16(t_acc + (uint32_t)tk, v);
              tmem_ld_wait();
              const uint32_t src = sbase + (uint32_t)((tk * BMW + row) * 4);
              float val[16];
              pld_add_f32x16<BMW * 4>(src, v, val);
              store_chunk(tk, val);
            }
          }
          return;
        }
        const bool main_lane = warp == EPI_WARP0 && lane == 0;
        const size_t slot_f = (size_t)ntok * BMW;
        const int T0 = (c.n_tiles / (int)gridDim.x) * (int)gridDim.x;          // first left-over tile
        float* mine = c.partials + ((size_t)(t - T0) + (c.sk_atomic ? 0 : blockIdx.x)) * slot_f;
        if (pair_send) {
          // (the second block of a pair: its "slot" is the first block's rings, once they are idle)
          if (!pmbar_wait_cluster(px_ready, 0, abort_flag)) { failed = true; return; }
          mine = ppeer_generic(smem, 0u);
        }
        for (int ch = ch0; ch < ntok / EPI_TOK; ch += chs) {
          uint32_t v[32];
          tmem_ld32(t_acc + (uint32_t)(ch * EPI_TOK), v);
          tmem_ld_wait();
          if (chs == 1) release_after(ch);                     // the accumulator is free for the next segment
          float* dst = mine + (size_t)(ch * EPI_TOK) * BMW + row;
          if (pair_send) {
#pragma unroll
            for (int k = 0; k < 32; ++k) dst[(size_t)k * BMW] = __uint_as_float(v[k]);
          } else if (c.sk_atomic) {
#pragma unroll
            for (int k = 0; k < 32; ++k) atomicAdd(dst + (size_t)k * BMW, __uint_as_float(v[k]));
          } else {
#pragma unroll
            for (int k = 0; k < 32; ++k) __stcg(dst + (size_t)k * BMW, __uint_as_float(v[k]));
          }
        }
        if (pair_send) {
          __syncwarp();
          if (lane == 0) {
            asm volatile("fence.acq_rel.cluster;" ::: "memory");
            pmbar_arrive_peer(ppeer_addr(px_done, 0u));
          }
          return;
        }
        __threadfence();                                       // this thread's part is in place before ...
        if (!(chs == 1 ? epi_sync() : help_sync())) { failed = true; return; }
        const long U = (long)(c.n_tiles - T0) * c.n_kb, Bn = (long)gridDim.x < U ? (long)gridDim.x : U;
        const long tu = (long)(t - T0) * c.n_kb;                               // the tile's first left-over unit
        const int first = sk_owner(tu, Bn, U), last = sk_owner(tu + c.n_kb - 1, Bn, U);
        if (main_lane) {
          const int arrived = atomicAdd(&c.counters[t], 1);    // ... the block's arrival shows
          *last_flag = arrived == last - first;
          __threadfence();
        }
        if (!(chs == 1 ? epi_sync() : help_sync())) { failed = true; return; }
        if (*last_flag) {
          const float* base = c.partials + ((size_t)(t - T0) + (c.sk_atomic ? 0 : first)) * slot_f;
          const int parts = c.sk_atomic ? 1 : last - first + 1;
          // 16 tokens at a time, the loads of two slots in flight together (what the registers of a thread hold)
          for (int tk = 16 * ch0; tk < ntok; tk += 16 * chs) {
            float val[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) val[k] = 0.f;
            const float* src = base + (size_t)tk * BMW + row;
            for (int s2 = 0; s2 < parts; s2 += 2) {
              const bool two = s2 + 1 < parts;
              float a[16], b[16];
#pragma unroll
              for (int k = 0; k < 16; ++k) a[k] = __ldcg(src + (size_t)s2 * slot_f + (size_t)k * BMW);
#pragma unroll
              for (int k = 0; k < 16; ++k) b[k] = two ? __ldcg(src + (size_t)(s2 + 1) * slot_f + (size_t)k * BMW) : 0.f;
#pragma unroll
              for (int k = 0; k < 16; ++k) val[k] = (val[k] + a[k]) + b[k];
            }
            store_chunk(tk, val);
          }
          if (main_lane) c.counters[t] = 0;              // ready for the next call
        }
      }
  };

  if (warp == 0) {
    // ===================================================================== activations by TMA
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");   // the activations may come from the preceding kernel
      int s = 0; uint32_t par = 1; int jb = 0;             // box slot, parity of its previous use, boxes so far
      SegIter si; si.init(c, blockIdx.x, gridDim.x);
      Seg sg;
      while (!failed && si.next(sg)) {
        const int tt = sg.tile % c.n_ttiles;
        KWalk kw;
        if (HEADS) kw.start(c, sg.kb0);
        for (int kb = sg.kb0; kb < sg.kb1 && !failed; ++kb) {
          const int xcol = HEADS ? kw.xcol(c) : kb * BK;
          if (HEADS) kw.step(c, 1);
          const int h_lo = sg.half < 0 ? 0 : sg.half, h_hi = sg.half < 0 ? c.nh : sg.half + 1;
          for (int h = h_lo; h < h_hi; ++h, ++jb) {
            if (jb >= BSLOTS && !pmbar_wait(empty_b + 8 * s, par, abort_flag, true)) { failed = true; break; }
            const uint32_t fb = full_b + 8 * s;
            pmbar_expect_tx(fb, (uint32_t)(c.bn * BK * 2));
            // (a box that starts at or beyond the last token is all zeros: the tensor map ends at M)
            tma_box2(sbase + B_RING + s * B_BYTES, &c.xmap, xcol, (tt * c.nh + h) * c.bn, fb);
            if (++s == BSLOTS) { s = 0; par ^= 1; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issue
    if (lane == 0) {
      int s = 0; uint32_t par = 0; int tcount = 0;         // weight stage and its parity
      int sb = 0; uint32_t parb = 0;                       // activation box slot and its parity
      SegIter si; si.init(c, blockIdx.x, gridDim.x);
      Seg sg;
      for (; !failed && si.next(sg); ++tcount) {
        // A tile of one box alternates between the two accumulators; a tile of two boxes holds both: the
        // de-quantised weight stage then serves 512 tokens, and the accumulator of the first 256 is drained by
        // the epilogue while the MMAs of the next tile already run on ... once it is free again (per-accumulator waits).
        const int acc0 = c.nh == 2 ? 0 : (tcount & 1);
        const int au = c.nh == 2 ? tcount : (tcount >> 1);   // earlier tiles that used this tile's accumulator(s)
        const int h_lo = sg.half < 0 ? 0 : sg.half, h_hi = sg.half < 0 ? c.nh : sg.half + 1;   // (a half tile is a block's last)
        for (int kb = sg.kb0; kb < sg.kb1 && !failed; ++kb) {
          if (!pmbar_wait(full_a + 8 * s, par, abort_flag)) { failed = true; break; }
          const uint64_t adesc = smem_desc_sw128(sbase + s * A_BYTES);
          for (int h = h_lo; h < h_hi; ++h) {
            if (kb == sg.kb0 && au >= 1 && !pmbar_wait(acc_empty + 8 * (acc0 + h), (au - 1) & 1, abort_flag)) { failed = true; break; }
            // (bf16: the de-quantisers waited for the activation box themselves and converted it)
            if (!CONV && !pmbar_wait(full_b + 8 * sb, parb, abort_flag)) { failed = true; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)((acc0 + h) * MAXBN);
            const uint64_t bdesc = smem_desc_sw128(sbase + B_RING + sb * B_BYTES);
#pragma unroll
            for (int k16 = 0; k16 < BK / 16; ++k16)     // 32 bytes along K per MMA: +2 in the address field
              umma_f16(d_tmem, adesc + 2 * k16, bdesc + 2 * k16, c.idesc, (kb > sg.kb0 || k16 > 0) ? 1u : 0u);
            umma_commit(empty_b + 8 * sb);              // the box is free once these MMAs have read it
            if (++sb == BSLOTS) { sb = 0; parb ^= 1; }
          }
          if (failed) break;
          umma_commit(empty_a + 8 * s);                 // ... and the weight stage after the last of them
          if (++s == PSTAGES) { s = 0; par ^= 1; }
        }
        if (failed) break;
        for (int h = h_lo; h < h_hi; ++h) umma_commit(acc_full + 8 * (acc0 + h));
        // (the de-quantiser warps that help with the last segment's epilogue cannot follow the phases of the
        //  accumulator barriers -- a parity wait cannot tell "not yet" from "two phases ago" -- so the last
        //  segment completes a barrier of its own, which has this one phase)
        SegIter peek = si;
        Seg nxt;
        if (!peek.next(nxt)) umma_commit(last_full);
      }
      if (c.pair_split && crank == 0 && !failed) {
        // the first block of a pair: once its own MMAs are complete nothing reads its rings any more
        if (pmbar_wait(last_full, 0, abort_flag)) {
          asm volatile("fence.acq_rel.cluster;" ::: "memory");
          pmbar_arrive_peer(ppeer_addr(px_ready, 1u));
        } else {
          failed = true;
        }
      }
    }
  } else if (warp >= DQ_WARP0) {
    // ===================================================================== de-quantisers
    // Two teams of six warps take alternate stages (a team always meets the same ring slots again, so its parity
    // waits are never more than one phase away from their barriers); a thread converts 32 codes of a weight row,
    // the first 64 threads of a team a second such item (256 items on 192 threads).  The teams are the twelve
    // warps on the three schedulers that do NOT host the MMA warp (warp % 4 != 1): the lane that issues the MMAs
    // runs one dependent instruction after the other, and with four busy warps on its scheduler every one of them
    // waited longer for its issue slot (measured with those four warps idle, results wrong by construction: Qwen
    // gate at M = 2048 296 -> 266 us with tiles of 256 tokens, 251 -> 232 us with 512).  The four warps 9, 13, 17,
    // 21 only help with the block's last epilogue (below).
    const int sc = warp & 3;
    if (sc != 1) {
    const int pos = ((warp - DQ_WARP0) >> 2) * 3 + (sc == 0 ? 0 : sc - 1);      // 0..11 among the twelve
    const int team = pos / DQ_TEAM_WARPS;
    const int dt = (pos - team * DQ_TEAM_WARPS) * 32 + lane;                    // 0..191
    constexpr int TEAM_TH = DQ_TEAM_WARPS * 32;
    const int n_items = dt + TEAM_TH < 2 * BMW ? 2 : 1;                         // items dt and dt + 192 of 256
    const int G = p.K / kGroup;
    int done = 0;                      // stage iterations before this segment
    constexpr bool heads = HEADS;
    SegIter si; si.init(c, blockIdx.x, gridDim.x);
    Seg sg;
    for (; !failed && si.next(sg); done += sg.kb1 - sg.kb0) {
      const int it0 = done - sg.kb0;   // stage iteration of k-block kb of this segment = it0 + kb
      const int wt = sg.tile / c.n_ttiles;
      const int jn = job_of_wt(wt);
      const JobDev& jb = p.job[jn];
      bool live[2];
      const uint8_t* wrow[2];
      const __half* srow[2];
      const __half* zrow[2];
      uint32_t st_off[2];              // row and half of the item inside a stage (the swizzle is applied per word)
      int hf_of[2], r7[2];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const int item = dt + m * TEAM_TH;
        const int r = (item >> 1) & (BMW - 1), hf = item & 1;
        const RowInfo ri = tile_row(jb, wt - c.wtile_begin[jn], r);
        live[m] = m < n_items && ri.stored >= 0;
        const JobDev& src = (jb.pair == 1 && (r & 1)) ? p.job[jn + 1] : jb;    // odd rows of a SwiGLU pair: the up matrix
        wrow[m] = src.w + (size_t)(live[m] ? ri.stored : 0) * (p.K / 2) + hf * 16;
        srow[m] = src.scales + (size_t)(live[m] ? ri.stored : 0) * G;
        zrow[m] = src.zeros + (size_t)(live[m] ? ri.stored : 0) * G;
        st_off[m] = (uint32_t)(r * 128);
        hf_of[m] = hf; r7[m] = r & 7;
      }
      const int kb0 = ((done & 1) == team) ? sg.kb0 : sg.kb0 + 1;
      // codes and scale / zero-point of this team's next k-block are kept in registers
      uint4 q0[2];
      __half s0[2], z0[2];
#pragma unroll
      for (int m = 0; m < 2; ++m) { q0[m] = make_uint4(0, 0, 0, 0); s0[m] = __ushort_as_half(0); z0[m] = s0[m]; }
      // codes, scale and zero-point of visited k-block v of an item's row; `valid` channels of it are kept
      // (a leading block needs no mask: the activation tensor map ends at k_in, so the tail of its last k-block
      //  meets zeros)
      // (the stored k-block of a visited one costs a division with per-head maps: worked out once for both items)
      auto fetch = [&](int m, int stored, uint4& q, __half& sc2, __half& zr) {
        q = __ldg(reinterpret_cast<const uint4*>(wrow[m] + (size_t)stored * 32));
        sc2 = __ldg(srow[m] + (stored >> 1)); zr = __ldg(zrow[m] + (stored >> 1));
      };
      KWalk kw;                                            // this team's current k-block
      if (heads && kb0 < sg.kb1) kw.start(c, kb0);
      if (kb0 < sg.kb1) {
        const int st0 = heads ? kw.stored(c) : kb0;
#pragma unroll
        for (int m = 0; m < 2; ++m)
          if (live[m]) fetch(m, st0, q0[m], s0[m], z0[m]);
      }
      for (int kb = kb0; kb < sg.kb1; kb += 2) {
        const int it = it0 + kb;
        const int s = it & (PSTAGES - 1);
        const uint32_t use = (uint32_t)(it / PSTAGES);
        uint4 q1[2];
        __half s1[2], z1[2];
        const bool more = kb + 2 < sg.kb1;
        const int v0 = heads ? kw.valid(c) : BK;           // kept channels of this k-block
        if (heads) kw.step(c, 2);
        const int st1 = (heads && more) ? kw.stored(c) : kb + 2;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          q1[m] = make_uint4(0, 0, 0, 0); s1[m] = s0[m]; z1[m] = z0[m];
          if (live[m] && more) fetch(m, st1, q1[m], s1[m], z1[m]);
        }
        if (it >= PSTAGES && !pmbar_wait(empty_a + 8 * s, (use - 1) & 1, abort_flag)) { failed = true; break; }
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          if (m >= n_items) break;
          const uint32_t a_st = sbase + s * A_BYTES + st_off[m];
          const __half2 sh2 = __half2half2(s0[m]);
          const __half2 cz2 = __float2half2_rn((8.f - __half2float(z0[m])) * __half2float(s0[m]));
          const uint32_t qw[4] = {q0[m].x, q0[m].y, q0[m].z, q0[m].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            // (eight channels per word; keep counts are multiples of eight, so a word is kept or pruned whole)
            const uint4 o = (live[m] && (!HEADS || hf_of[m] * 32 + j * 8 < v0)) ? dequant_word(qw[j], sh2, cz2) : make_uint4(0, 0, 0, 0);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a_st + (uint32_t)(((hf_of[m] * 4 + j) ^ r7[m]) * 16)), "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w) : "memory");
          }
        }
        if constexpr (CONV) {
          // bf16 activations: the tensor cores run on fp16 (8 more mantissa bits for the weights than bf16
          // would leave them); the activation tile that TMA delivered is converted in place
          for (int h = 0; h < c.nh && !failed; ++h) {
            const int jb2 = it * c.nh + h;                 // the k-block's boxes in the order the producer issued them
            const int sb = jb2 % BSLOTS;
            if (!pmbar_wait(full_b + 8 * sb, (uint32_t)(jb2 / BSLOTS) & 1, abort_flag)) { failed = true; break; }
            const uint32_t b_st = sbase + B_RING + sb * B_BYTES;
            for (int ci = dt; ci < c.bn * 8; ci += TEAM_TH) {
              uint32_t v0, v1, v2, v3;
              asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(b_st + ci * 16));
              v0 = bf16x2_to_f16x2(v0); v1 = bf16x2_to_f16x2(v1); v2 = bf16x2_to_f16x2(v2); v3 = bf16x2_to_f16x2(v3);
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(b_st + ci * 16), "r"(v0), "r"(v1), "r"(v2), "r"(v3) : "memory");
            }
          }
          if (failed) break;
        }
        fence_async_smem();            // generic-proxy writes must be visible to the tensor core (async proxy)
        __syncwarp();
        if (lane == 0) pmbar_arrive(full_a + 8 * s);
#pragma unroll
        for (int m = 0; m < 2; ++m) { q0[m] = q1[m]; s0[m] = s1[m]; z0[m] = z1[m]; }
      }
    }
    }
    // the block's segments, counted by every warp of this group (the idle four included)
    Seg last_sg = {0, 0, 0, -1};
    int n_seg = 0;
    {
      SegIter sj; sj.init(c, blockIdx.x, gridDim.x);
      Seg sgj;
      while (sj.next(sgj)) { last_sg = sgj; ++n_seg; }
    }
    // the block's last segment: this warp takes a fifth of its chunks beside the epilogue warp of its tensor-memory
    // quadrant (warps 8 + q, 12 + q, 16 + q, 20 + q: chunks 1, 2, 3, 4 of every five)
    if (c.helpers && !failed && n_seg > 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");   // outputs and workspace: after the preceding kernel
      if (!pmbar_wait(last_full, 0, abort_flag, true)) failed = true;
      if (!failed) epilogue_segment(last_sg, n_seg - 1, 1 + (warp - DQ_WARP0) / 4, 5, true);
    }
  } else if (warp >= EPI_WARP0) {
    // ===================================================================== epilogue
    asm volatile("griddepcontrol.wait;" ::: "memory");     // positions, outputs and workspace: after the preceding kernel
    int tcount = 0;
    SegIter si; si.init(c, blockIdx.x, gridDim.x);
    Seg sg;
    for (; !failed && si.next(sg); ++tcount) {
      // The block's last segment: nothing is left to overlap its epilogue with, and the sixteen de-quantiser warps
      // are idle by then, so the four of each tensor-memory quadrant take four fifths of its chunks.
      SegIter peek = si;
      Seg nxt;
      const bool helped = c.helpers && !peek.next(nxt);
      epilogue_segment(sg, tcount, 0, helped ? 5 : 1, false);
    }
  }

  if (failed && lane == 0) atomicExch(c.status, UNIQL_ERR_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
  if (c.pair_split) {                   // neither block of a pair leaves while the other may still send to it
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
}

// -------------------------------------------------------------------------------- host side
typedef CUresult (*PEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

PEncodeFn p_encoder() {
  static PEncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PEncodeFn>(ptr);
    else
      cudaGetLastError();
  });
  return fn;
}

int p_sm_count() {
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
    return v;
  return 148;
}

int host_job_tiles(const JobDev& j) {
  if (j.pair == 2) return 0;                                       // its rows ride in the tiles of the job before
  if (j.pair == 1) return (j.k_out + BMW / 2 - 1) / (BMW / 2);
  if (j.rope.enabled) return (j.rope.n_heads * (j.rope.head_keep / 2) + BMW / 2 - 1) / (BMW / 2);
  return (j.k_out + BMW - 1) / BMW;
}

template <typename T, bool CONV, bool HEADS>
int launch_pth(const Params& p, const PrefillCfg& c, int grid, cudaStream_t stream) {
  const size_t smem = 1024 + (size_t)RING_BYTES + 512;
  auto kern = prefill_kernel<T, CONV, HEADS>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return UNIQL_ERR_CUDA;
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(PTH);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = opt(kOptPdl) ? 1 : 0;
  if (c.pair_split) {
    // clusters of two, only when every pair can be resident at once; else the caller plans without them
    attr[lc.numAttrs].id = cudaLaunchAttributeClusterDimension;
    attr[lc.numAttrs].val.clusterDim.x = 2;
    attr[lc.numAttrs].val.clusterDim.y = 1;
    attr[lc.numAttrs].val.clusterDim.z = 1;
    ++lc.numAttrs;
    // (asked once per kernel instance: the answer depends on the block's resources, which do not change)
    static std::atomic<int> max_clusters{-1};
    int n_clusters = max_clusters.load();
    if (n_clusters < 0) {
      if (cudaOccupancyMaxActiveClusters(&n_clusters, kern, &lc) != cudaSuccess) { cudaGetLastError(); n_clusters = 0; }
      max_clusters.store(n_clusters);
    }
    if (n_clusters * 2 < grid) return UNIQL_ERR_UNSUPPORTED;
  }
  if (cudaLaunchKernelEx(&lc, kern, p, c) != cudaSuccess) { cudaGetLastError(); return c.pair_split ? UNIQL_ERR_UNSUPPORTED : UNIQL_ERR_CUDA; }
  return UNIQL_OK;
}
template <typename T, bool CONV>
int launch_pt(const Params& p, const PrefillCfg& c, int grid, cudaStream_t stream) {
  return c.km_period != 0 ? launch_pth<T, CONV, true>(p, c, grid, stream) : launch_pth<T, CONV, false>(p, c, grid, stream);
}

}  // namespace

// The tensor-core path takes: the leading k_in input channels (the hidden dimension D_h is never pruned,
// D_int is pruned as a leading block: Section 3.4) or one family of per-head kept blocks (the input side of
// o_proj / out_proj: heads on 64-channel boundaries, keep a multiple of 8), any output map, both activation types.
int prefill_supported(const Params& p) {
  if (p.M < 1) return 0;
  if (p.dt != UNIQL_F16 && p.dt != UNIQL_BF16) return 0;
  if (p.imap.n_fam != 1) return 0;
  {
    const Fam& a = p.imap.fam[0];
    if (a.count == 1) {
      if (a.start != 0) return 0;
    } else if ((a.start % BK) != 0 || (a.period % BK) != 0 || (a.keep % 8) != 0) {
      return 0;                    // per-head input maps: heads on k-block boundaries, 16-byte activation boxes
    }
  }
  if ((p.ldx % 8) != 0 || (((uintptr_t)p.x) & 15) != 0) return 0;       // TMA: 16-byte base and row pitch
  if ((p.K % kGroup) != 0) return 0;
  return 1;
}

int launch_prefill(const Params& p, const LaunchCfg& cfg) {
  PEncodeFn enc = p_encoder();
  if (!enc) return UNIQL_ERR_CUDA;
  if (!cfg.workspace || cfg.ws_bytes < decode_workspace_header_bytes()) return UNIQL_ERR_WORKSPACE;   // status word
  const int env_grid = opt(kOptPrefillGrid), env_streamk = opt(kOptPrefillStreamk);
  PrefillCfg c;
  memset(&c, 0, sizeof(c));
  c.bn = p.M <= 64 ? 64 : (p.M <= 128 ? 128 : 256);
  int wt = 0;
  for (int j = 0; j < p.n_jobs; ++j) { c.wtile_begin[j] = wt; wt += host_job_tiles(p.job[j]); }
  for (int j = p.n_jobs; j <= kMaxPJobs; ++j) c.wtile_begin[j] = wt;
  if (wt < 1) return UNIQL_ERR_SHAPE;
  {
    const Fam& a = p.imap.fam[0];
    c.km_start = a.start / BK;
    c.km_period = a.count > 1 ? a.period / BK : 0;
    c.km_keep = a.keep;
    c.km_kbh = (a.keep + BK - 1) / BK;
    c.n_kb = c.km_kbh * a.count;
  }
  const uint32_t fmt = 0u;      // both operands fp16 (bf16 activations are converted in shared memory)
  // instruction descriptor: fp32 accumulate, A and B of the activation type, both K-major, N = bn, M = 128
  c.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(c.bn >> 3) << 17) | ((uint32_t)(BMW >> 4) << 24);
  c.status = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(cfg.workspace) + decode_status_offset());
  const int sms = p_sm_count();
  // workspace: [header: counters, status][fp16 copy of bf16 activations][stream-K partial tiles]
  size_t ws_used = (decode_workspace_header_bytes() + 255) & ~(size_t)255;
  c.counters = reinterpret_cast<int*>(cfg.workspace);
  // bf16 activations: fp16 copy in the workspace when it fits (else converted tile by tile in the kernel)
  const void* xsrc = p.x;
  int ldxs = p.ldx;
  bool conv_in_kernel = false;
  __half* x16 = nullptr;              // fp16 copy to be written by the pre-pass
  int x16_ld = 0;
  if (p.dt == UNIQL_BF16) {
    // (a row pitch of whole 128-byte lines: a box row that straddles two lines costs a second L2 request, measured
    //  as 1.09 instead of 0.85 us per k-block on the Qwen2.5-7B down projection at 12312 of 18944 input channels)
    int ldo = (p.k_in + 63) / 64 * 64;
    const size_t off = ws_used;
    if (cfg.ws_bytes < off + (size_t)p.M * ldo * 2) ldo = (p.k_in + 7) / 8 * 8;
    const size_t need = off + (size_t)p.M * ldo * 2;
    if (cfg.ws_bytes >= need && opt(kOptPrefillConvert) != 1) {
      x16 = reinterpret_cast<__half*>(reinterpret_cast<unsigned char*>(cfg.workspace) + off);
      x16_ld = ldo;
      xsrc = x16;
      ldxs = ldo;
      ws_used = (need + 255) & ~(size_t)255;
    } else {
      conv_in_kernel = true;
    }
  }
  // The shape of the work: tokens per tile (one accumulator, or both = 512 tokens, so that a de-quantised weight
  // stage serves twice the tokens) and whether the tiles left over after the whole rounds are split along K.
  // Stream-K serves the tiles left over when whole tiles would leave SMs idle in their last round and the slots
  // of the parts fit in the workspace.  It pays when the k-blocks a block no longer waits for outweigh the
  // hand-over.  Measured on B200: a k-block takes about 0.65 us (1.07 us on both accumulators: 1.65 times the time
  // for twice the work); a hand-over at the end of a block (every tile split) 20 - 40 us, growing with the number
  // of blocks on a tile and the tile's width; a hand-over in front of whole tiles is hidden behind them unless a
  // tile has so many parts that reading them back (11 us per part of 256 tokens) outlasts the whole tiles.
  // Both tile widths are costed with these figures and the cheaper one runs: wide tiles win where they still fill
  // the SMs (Qwen2.5-7B gate at M = 512..4096: 17-22 % faster), narrow ones where wide tiles would leave most SMs
  // without a tile (q / o projections at M = 512) or push a few left-over tiles into a round of their own.
  int g2 = sms;
  if (env_grid >= 1 && env_grid <= sms) g2 = env_grid;            // tests: odd splits on small problems
  bool any_rope = false;
  for (int j = 0; j < p.n_jobs; ++j) any_rope = any_rope || p.job[j].rope.enabled != 0;
  struct Plan { int nh, ttiles, tiles, left; bool streamk, atomic, halves, pair; size_t sums; double us; };
  static std::atomic<bool> pair_refused{false};       // a cluster launch was refused once: planned without from then on
  auto plan_for = [&](int nh) {
    Plan q;
    q.nh = nh;
    const int ntok = c.bn * nh;
    q.ttiles = (p.M + ntok - 1) / ntok;
    const long tiles = (long)wt * q.ttiles;
    q.tiles = tiles <= (1 << 24) ? (int)tiles : (1 << 24);
    q.left = q.tiles % g2;
    const double kcost = nh == 2 ? 1.07 : 0.65;
    const double wide = ntok / 256.0;
    // blocks on the split tile with the most of them: its finishing block reads that many slots back
    const long units = (long)q.left * c.n_kb;
    const long bt = units < g2 ? units : g2;
    const double pmax = q.left ? (double)((bt + q.left - 1) / q.left + 1) : 0.0;
    double hand_over;
    q.atomic = false;
    // a k-block of a one-box tile by the number of busy SMs (0.45 us with 28 of them, 0.61 us with all)
    auto kb1 = [&](int busy) { return 0.42 + 0.19 * (busy < g2 ? busy : g2) / g2; };
    if (q.tiles < g2) {
      // every tile is split and every block ends on a split tile: the hand-over is shared with the de-quantiser warps
      // (one-box tiles, measured at M = 64 .. 512 on seven layer shapes: 5 us per 64 tokens of the tile)
      hand_over = nh == 2 ? 24.0 + 2.0 * pmax * wide : (14.0 + pmax) * wide;
    } else {
      // The split tiles come first and whole tiles follow.  Reading a tile's slots back takes the four epilogue
      // warps 11 us per slot of 256 tokens, and a split tile in front of whole tiles has three or more parts: that
      // outlasts the first whole tile, whose epilogue then waits (measured 37 us lost on the Qwen2.5-7B gate at keep
      // 0.65, M = 2048, three parts).  Here the parts are added into one sum per tile instead (reductions done in
      // L2): 14 us per 256 tokens, measured, most of it hidden behind the whole tiles.
      q.atomic = true;
      hand_over = 14.0 * wide;
    }
    // (a tile with the rotary epilogue costs its finishing block about twice as long: measured on the Qwen2.5-7B
    //  q|k launch at M = 2048, head dim 84, where the split forms lost 8 us against this estimate without it)
    if (any_rope) hand_over += 12.0 * wide;
    if (env_streamk == 1) q.atomic = false;                            // tests: the form of the hand-over forced
    if (env_streamk == 2) q.atomic = true;
    // (a split is taken where it is estimated 5 % ahead: its hand-over varies more than a whole tile's time)
    const double us_split = 1.05 * ((double)q.tiles / g2 * c.n_kb * ((nh == 1 && q.tiles < g2) ? kb1(g2) : kcost) + hand_over);
    // Whole tiles.  On both accumulators a k-block takes 0.84 us when every SM runs one and less when some have no
    // tile (0.79 us with 28 busy SMs: they share the activation traffic out of L2), and between two tiles of a block
    // the MMAs wait 7 - 10 us for the epilogue to drain the accumulators (in-kernel time stamps, Qwen2.5-7B gate at
    // M = 2048); fitted over 48 launches (16 shapes at M = 512, 1024, 2048, every width and hand-over forced in turn).
    const int rounds = (q.tiles + g2 - 1) / g2;
    double us_whole = (double)rounds * c.n_kb * kcost;
    if (nh == 1 && q.tiles <= g2) us_whole = c.n_kb * kb1(q.tiles);
    if (nh == 2)
      us_whole = (double)(q.tiles / g2) * c.n_kb * 0.96 + (q.left ? c.n_kb * (0.90 + 0.06 * q.left / g2) : 0.0) + 10.0 * (rounds - 1);
    // one fp32 slot per (left-over tile, block) piece, or one sum per left-over tile
    q.sums = (size_t)(q.atomic ? q.left : q.left + g2) * ntok * BMW * 4;
    const bool want = env_streamk >= 0 ? (env_streamk >= 1) : (q.left != 0 && us_split < us_whole);
    q.streamk = want && q.left != 0 && cfg.ws_bytes >= ws_used + q.sums && q.tiles <= (1 << 16);
    q.us = q.streamk ? us_split : us_whole;
    // Tiles of two boxes left over after the whole rounds, when they are few: each runs as two half tiles (one box,
    // 256 tokens) on two blocks, a block's last segment -- no hand-over, and the round takes a one-box tile's time
    // (0.45 - 0.6 us per k-block by the number of busy SMs) instead of a two-box tile's on a few SMs.
    q.halves = false;
    if (nh == 2 && q.left != 0 && 2 * q.left <= g2 && q.tiles > g2 && !conv_in_kernel && env_streamk < 1 && opt(kOptPrefillDual) != 2) {
      const double us_halves = (double)(q.tiles / g2) * (c.n_kb * 0.96 + 10.0) + c.n_kb * (0.45 + 0.15 * 2 * q.left / g2);
      if (us_halves < q.us || opt(kOptPrefillDual) == 3) { q.halves = true; q.streamk = false; q.us = us_halves; }
    }
    // Few tiles of one box (at most one for every two SMs): a cluster of two blocks per tile, half of the
    // contraction each, the second block's sums handed over through the first one's shared memory (about 5 us
    // against the 11 - 28 us of a hand-over through the workspace; a k-block takes the same 0.5 - 0.65 us).
    q.pair = false;
    if (nh == 1 && 2 * q.tiles <= sms && c.n_kb >= 4 && env_grid == 0 && !pair_refused.load() && (env_streamk < 0 || env_streamk == 3)) {
      const double us_pair = (double)(c.n_kb - c.n_kb / 2) * kb1(2 * q.tiles) + 1.0 + 4.5 * wide + (any_rope ? 3.0 : 0.0);
      // (against a split over all SMs it has to be 10 % ahead: with long contractions the two come out level and
      //  the split measured ahead, Qwen2.5-7B down projection at M = 512)
      if (us_pair * (q.streamk ? 1.10 : 1.0) < q.us || env_streamk == 3) { q.pair = true; q.streamk = false; q.us = us_pair; }
    }
    return q;
  };
  Plan pl = plan_for(1);
  {
    // -1: by cost, 0: never, 1: wherever M > 256; tests: 2 the same without half tiles, 3 with them wherever they fit
    const int dual = opt(kOptPrefillDual);
    if (p.M > MAXBN && dual != 0) {
      const Plan p2 = plan_for(2);
      if (dual >= 1 || p2.us < pl.us) pl = p2;
    }
  }
  c.helpers = opt(kOptPrefillHelpers) != 0;
  c.nh = pl.nh;
  c.halves = pl.halves ? 1 : 0;
  c.pair_split = pl.pair ? 1 : 0;
  c.n_ttiles = pl.ttiles;
  c.n_tiles = pl.tiles;
  if ((long)wt * pl.ttiles > (1 << 24)) return UNIQL_ERR_SHAPE;
  int grid = c.n_tiles < g2 ? c.n_tiles : g2;
  if (pl.pair) grid = 2 * c.n_tiles;
  {
    if (pl.streamk) {
      c.streamk = 1;
      c.sk_atomic = pl.atomic ? 1 : 0;
      c.partials = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(cfg.workspace) + ws_used);
      grid = g2;
      // (slots are written before they are read; sums start at zero)
      if (pl.atomic && cudaMemsetAsync(c.partials, 0, pl.sums, cfg.stream) != cudaSuccess) return UNIQL_ERR_CUDA;
    }
    if (x16) {
      const long units = (long)p.M * (x16_ld / 8);
      long blocks = (units + 255) / 256;
      if (blocks > (long)sms * 8) blocks = (long)sms * 8;
      cudaLaunchConfig_t lc;
      memset(&lc, 0, sizeof(lc));
      lc.gridDim = dim3((unsigned)blocks);
      lc.blockDim = dim3(256);
      lc.stream = cfg.stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      lc.attrs = attr;
      lc.numAttrs = opt(kOptPdl) ? 1 : 0;
      if (cudaLaunchKernelEx(&lc, x_to_f16_kernel, reinterpret_cast<const __nv_bfloat16*>(p.x), p.ldx, p.M, p.k_in, x16, x16_ld) != cudaSuccess) {
        cudaGetLastError();
        return UNIQL_ERR_CUDA;
      }
    }
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)p.k_in, (cuuint64_t)p.M};
    const cuuint64_t strides[1] = {(cuuint64_t)ldxs * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)c.bn};
    const cuuint32_t es[2] = {1, 1};
    const CUresult r = enc(&c.xmap, conv_in_kernel ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16,
                           2, const_cast<void*>(xsrc), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return UNIQL_ERR_CUDA;
  }
  int rc;
  if (p.dt == UNIQL_BF16)
    rc = conv_in_kernel ? launch_pt<__nv_bfloat16, true>(p, c, grid, cfg.stream)
                        : launch_pt<__nv_bfloat16, false>(p, c, grid, cfg.stream);
  else
    rc = launch_pt<__half, false>(p, c, grid, cfg.stream);
  if (rc == UNIQL_ERR_UNSUPPORTED && c.pair_split) {
    // the pairs cannot all be resident (or clusters cannot be launched here): planned again without them
    pair_refused.store(true);
    return launch_prefill(p, cfg);
  }
  return rc;
}

size_t prefill_workspace_bytes(int M, int K) {
  // status word and counters (shared header) + room for the fp16 copy of bf16 activations + the slots of tiles
  // split along K: fewer than two per SM, of 256 tokens, or of 512 where tiles take both accumulators
  return ((decode_workspace_header_bytes() + 255) & ~(size_t)255) + (size_t)M * ((K + 63) / 64 * 64) * 2 + 256 +
         (size_t)2 * p_sm_count() * (M > MAXBN ? 2 * MAXBN : MAXBN) * BMW * 4;
}

}  // namespace uniql
