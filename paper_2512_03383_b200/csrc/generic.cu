// Generic kernel of the pruned 4-bit linear layer: any M, any channel map, optional
// rotary epilogue.  A plain shared-memory tiled contraction on the CUDA cores in fp32;
// it exists for the shapes the specialised kernels do not take (17 <= M < 64, unaligned
// maps) and as an A/B partner in tests.  Not a CPU fallback: it is a CUDA kernel.
#include "common.cuh"

namespace uniql {
namespace {

constexpr int BM = 64, BN = 64, BK = 32, NT = 256;

// Column c of a tile -> (stored weight row, compact output column).  In rope mode a tile
// holds 32 rotation pairs: columns 0..31 are the first-half members, 32..63 their partners.
struct ColInfo { int stored; int out; int pair_p; int kvh; };

__device__ inline ColInfo resolve_col(const JobDev& jb, int tile, int c) {
  ColInfo ci;
  ci.pair_p = -1; ci.kvh = 0;
  if (jb.rope.enabled) {
    int half = jb.rope.head_keep >> 1;
    int P = tile * (BN / 2) + (c & (BN / 2 - 1));
    int hi = c >= BN / 2;
    int np = jb.rope.n_heads * half;
    if (P >= np) { ci.stored = -1; ci.out = -1; return ci; }
    int h = P / half, cc = P - h * half;
    ci.stored = h * jb.rope.head_dim + hi * (jb.rope.head_dim >> 1) + cc;
    ci.out = h * jb.rope.head_keep + hi * half + cc;
    ci.pair_p = cc;
    ci.kvh = h / jb.rope.rep;
  } else {
    int j = tile * BN + c;
    if (j >= jb.k_out) { ci.stored = -1; ci.out = -1; return ci; }
    ci.stored = map_compact_to_stored(jb.omap, j);
    ci.out = j;
  }
  return ci;
}

template <typename T>
__global__ void __launch_bounds__(NT) generic_kernel(const __grid_constant__ Params p, int4 tile_begin) {
  __shared__ float xs[BK][BM + 1];
  __shared__ float wsm[BK][BN + 1];
  __shared__ int s_stored[BN], s_out[BN], s_pp[BN], s_kvh[BN];
  __shared__ int s_kmap[BK];
  __shared__ float tile_out[BM][BN + 1];

  // which job does this column tile belong to?
  int bt = blockIdx.x;
  int jn = 0;
  const int tb[4] = {tile_begin.x, tile_begin.y, tile_begin.z, tile_begin.w};
  while (jn + 1 < p.n_jobs && bt >= tb[jn + 1]) ++jn;
  const JobDev& jb = p.job[jn];
  const int tile = bt - tb[jn];
  const int m0 = blockIdx.y * BM;
  const int tid = threadIdx.x;

  if (tid < BN) {
    ColInfo ci = resolve_col(jb, tile, tid);
    s_stored[tid] = ci.stored; s_out[tid] = ci.out; s_pp[tid] = ci.pair_p; s_kvh[tid] = ci.kvh;
  }
  const T* x = reinterpret_cast<const T*>(p.x);
  const int G = p.K / kGroup;
  const int tx = tid & 15, ty = tid >> 4;     // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < p.k_in; k0 += BK) {
    __syncthreads();
    if (tid < BK) s_kmap[tid] = (k0 + tid < p.k_in) ? map_compact_to_stored(p.imap, k0 + tid) : -1;
    for (int e = tid; e < BK * BM; e += NT) {           // x tile, k fastest for coalescing
      int mm = e / BK, kk = e - mm * BK;
      float v = 0.f;
      if (m0 + mm < p.M && k0 + kk < p.k_in) v = DT<T>::to_f(x[(size_t)(m0 + mm) * p.ldx + k0 + kk]);
      xs[kk][mm] = v;
    }
    __syncthreads();
    for (int e = tid; e < BK * BN; e += NT) {
      int c = e / BK, kk = e - c * BK;
      int sk = s_kmap[kk], sr = s_stored[c];
      float w = 0.f;
      if (sk >= 0 && sr >= 0) {
        uint8_t byte = jb.w[(size_t)sr * (p.K / 2) + (sk >> 1)];
        int code = (sk & 1) ? (byte >> 4) : (byte & 15);
        float s = __half2float(jb.scales[(size_t)sr * G + sk / kGroup]);
        float z = __half2float(jb.zeros[(size_t)sr * G + sk / kGroup]);
        w = s * ((float)code - z);
      }
      wsm[kk][c] = w;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = xs[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = wsm[kk][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
  }
  // bias, then park the fp32 tile in shared memory so that rotation partners can meet
  const T* bias = reinterpret_cast<const T*>(jb.bias);
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int c = tx + 16 * j;
      float v = acc[i][j];
      if (bias && s_stored[c] >= 0) v += DT<T>::to_f(bias[s_stored[c]]);
      tile_out[ty * 4 + i][c] = v;
    }
  __syncthreads();
  T* y = reinterpret_cast<T*>(jb.y);
  if (jb.rope.enabled) {
    int half = jb.rope.head_keep >> 1;
    for (int e = tid; e < BM * (BN / 2); e += NT) {
      int mm = e / (BN / 2), c = e - mm * (BN / 2);
      int m = m0 + mm;
      if (m >= p.M || s_out[c] < 0) continue;
      int pidx = p.idx[s_kvh[c] * half + s_pp[c]];
      pidx = min(max(pidx, 0), (jb.rope.head_dim >> 1) - 1);
      float cs, sn;
      rope_cos_sin(p.pos[m], p.rope_turn[pidx], cs, sn);
      float a = tile_out[mm][c], b = tile_out[mm][c + BN / 2];
      y[(size_t)m * jb.ldy + s_out[c]] = DT<T>::from_f(a * cs - b * sn);
      y[(size_t)m * jb.ldy + s_out[c + BN / 2]] = DT<T>::from_f(b * cs + a * sn);
    }
  } else {
    for (int e = tid; e < BM * BN; e += NT) {
      int mm = e / BN, c = e - mm * BN;
      int m = m0 + mm;
      if (m >= p.M || s_out[c] < 0) continue;
      y[(size_t)m * jb.ldy + s_out[c]] = DT<T>::from_f(tile_out[mm][c]);
    }
  }
}

}  // namespace

int launch_generic(const Params& p, const LaunchCfg& cfg) {
  int tb[5] = {0, 0, 0, 0, 0};
  for (int j = 0; j < p.n_jobs; ++j) {
    int tiles;
    if (p.job[j].rope.enabled) {
      int np = p.job[j].rope.n_heads * (p.job[j].rope.head_keep / 2);
      tiles = (np + BN / 2 - 1) / (BN / 2);
    } else {
      tiles = (p.job[j].k_out + BN - 1) / BN;
    }
    tb[j + 1] = tb[j] + tiles;
  }
  for (int j = p.n_jobs; j < 4; ++j) tb[j + 1] = tb[p.n_jobs];
  dim3 grid(tb[p.n_jobs], (p.M + BM - 1) / BM);
  if (grid.y > 65535) return UNIQL_ERR_SHAPE;
  int4 tbv = make_int4(tb[0], tb[1], tb[2], tb[3]);
  if (p.dt == UNIQL_F16)
    generic_kernel<__half><<<grid, NT, 0, cfg.stream>>>(p, tbv);
  else
    generic_kernel<__nv_bfloat16><<<grid, NT, 0, cfg.stream>>>(p, tbv);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

}  // namespace uniql
