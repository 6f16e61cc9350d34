// Storage helpers: nibble pack / unpack (bit-exact integer work) and a diagnostic full
// de-quantisation.  Memory-bound element-wise kernels with 128-bit accesses where the
// sizes allow.
#include "common.cuh"

namespace uniql {
namespace {

// two codes per byte, even input channel in the low nibble
__global__ void pack_kernel(const uint8_t* __restrict__ codes, uint8_t* __restrict__ packed, int64_t n_bytes) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n_bytes; i += stride) {
    uchar2 c = reinterpret_cast<const uchar2*>(codes)[i];
    packed[i] = (uint8_t)((c.x & 15) | (c.y << 4));
  }
}

__global__ void unpack_kernel(const uint8_t* __restrict__ packed, uint8_t* __restrict__ codes, int64_t n_bytes) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n_bytes; i += stride) {
    uint8_t b = packed[i];
    reinterpret_cast<uchar2*>(codes)[i] = make_uchar2(b & 15, b >> 4);
  }
}

template <typename T>
__global__ void dequant_kernel(const uint8_t* __restrict__ packed, const __half* __restrict__ scales,
                               const __half* __restrict__ zeros, int64_t N, int64_t K, T* __restrict__ w) {
  int64_t n_bytes = N * (K / 2);
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t G = K / kGroup;
  for (; i < n_bytes; i += stride) {
    int64_t n = i / (K / 2), b = i - n * (K / 2);
    int64_t g = (2 * b) / kGroup;
    float s = __half2float(scales[n * G + g]), z = __half2float(zeros[n * G + g]);
    uint8_t byte = packed[i];
    w[n * K + 2 * b] = DT<T>::from_f(s * ((float)(byte & 15) - z));
    w[n * K + 2 * b + 1] = DT<T>::from_f(s * ((float)(byte >> 4) - z));
  }
}

// Rows ids[m] of a 4-bit table, de-quantised: one block per (token, slice of the row), a thread per packed
// 32-bit word (eight channels, one 16-byte store).
template <typename T>
__global__ void embed_kernel(const uint8_t* __restrict__ packed, const __half* __restrict__ scales,
                             const __half* __restrict__ zeros, int64_t V, int64_t K, const int32_t* __restrict__ ids,
                             T* __restrict__ out, int64_t ldo, int* __restrict__ bad) {
  const int64_t m = blockIdx.y;
  int64_t row = ids[m];
  const bool in_range = row >= 0 && row < V;
  if (!in_range) {
    if (bad && threadIdx.x == 0 && blockIdx.x == 0) atomicExch(bad, 1);
    row = 0;                                   // the output row is zero-filled below
  }
  const int64_t words = K / 8, G = K / kGroup;
  const uint32_t* wrow = reinterpret_cast<const uint32_t*>(packed + row * (K / 2));
  for (int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; w < words; w += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t q = in_range ? __ldg(wrow + w) : 0u;
    const int64_t g = (w * 8) / kGroup;
    const float s = in_range ? __half2float(scales[row * G + g]) : 0.f;
    const float z = __half2float(zeros[row * G + g]);
    __align__(16) T v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = DT<T>::from_f(s * ((float)((q >> (4 * e)) & 15u) - z));
    T* o = out + m * ldo + w * 8;
    if ((reinterpret_cast<uintptr_t>(o) & 15) == 0) {
      *reinterpret_cast<uint4*>(o) = *reinterpret_cast<const uint4*>(v);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = v[e];
    }
  }
}

// Activations re-laid with every kept block padded to a multiple of 8 channels (zeros in the padding): the fast
// kernels read activations in 16-byte units, which blocks of 108 or 84 channels (multiples of 4) do not give.
// One thread per 4 output channels (8 bytes); x needs 2-byte alignment only.
__global__ void relay_x_kernel(const unsigned short* __restrict__ x, long long ldx, int M, int count, int keep, int keep8,
                               unsigned short* __restrict__ out) {
  // (programmatic dependent launch: the kernel behind this one may set itself up meanwhile; this one waits for its
  //  own predecessor before it reads x or overwrites the copy that predecessor may still read)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int units_row = count * (keep8 >> 2);
  const long long total = (long long)M * units_row;
  const bool vec = ((ldx & 3) == 0) && ((((uintptr_t)x) & 7) == 0) && ((keep & 3) == 0);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / units_row), u = (int)(i - (long long)m * units_row);
    const int h = u / (keep8 >> 2), r = (u - h * (keep8 >> 2)) * 4;
    const unsigned short* src = x + (size_t)m * ldx + (size_t)h * keep + r;
    uint2 v = make_uint2(0u, 0u);
    if (vec && r + 4 <= keep) {
      v = *reinterpret_cast<const uint2*>(src);
    } else {
      unsigned short e[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) e[k] = r + k < keep ? src[k] : (unsigned short)0;
      v.x = (uint32_t)e[0] | ((uint32_t)e[1] << 16);
      v.y = (uint32_t)e[2] | ((uint32_t)e[3] << 16);
    }
    *reinterpret_cast<uint2*>(out + (size_t)m * ((size_t)count * keep8) + (size_t)h * keep8 + r) = v;
  }
}

inline int grid_for(int64_t n, int threads) {
  static const int sms = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      return v;
    return 148;
  }();
  int64_t b = (n + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > (int64_t)sms * 16) b = (int64_t)sms * 16;
  return (int)b;
}

}  // namespace
}  // namespace uniql

int uniql::launch_relay_x(const void* x, long long ldx, int M, int count, int keep, int keep8, void* out, cudaStream_t stream) {
  const int64_t units = (int64_t)M * count * (keep8 / 4);
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3((unsigned)grid_for(units, 256));
  lc.blockDim = dim3(256);
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = opt(kOptPdl) ? 1 : 0;
  if (cudaLaunchKernelEx(&lc, relay_x_kernel, reinterpret_cast<const unsigned short*>(x), ldx, M, count, keep, keep8,
                         reinterpret_cast<unsigned short*>(out)) != cudaSuccess) {
    cudaGetLastError();
    return UNIQL_ERR_CUDA;
  }
  return UNIQL_OK;
}

using namespace uniql;

extern "C" int uniql_pack_u4(const uint8_t* codes, int64_t N, int64_t K, uint8_t* packed, void* stream) {
  if (!codes || !packed) return UNIQL_ERR_NULL;
  if (N < 0 || K < 0 || (K & 1)) return UNIQL_ERR_SHAPE;
  if (((uintptr_t)codes) & 1) return UNIQL_ERR_ALIGN;
  int64_t nb = N * (K / 2);
  if (nb == 0) return UNIQL_OK;
  pack_kernel<<<grid_for(nb, 256), 256, 0, (cudaStream_t)stream>>>(codes, packed, nb);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

extern "C" int uniql_unpack_u4(const uint8_t* packed, int64_t N, int64_t K, uint8_t* codes, void* stream) {
  if (!codes || !packed) return UNIQL_ERR_NULL;
  if (N < 0 || K < 0 || (K & 1)) return UNIQL_ERR_SHAPE;
  if (((uintptr_t)codes) & 1) return UNIQL_ERR_ALIGN;
  int64_t nb = N * (K / 2);
  if (nb == 0) return UNIQL_OK;
  unpack_kernel<<<grid_for(nb, 256), 256, 0, (cudaStream_t)stream>>>(packed, codes, nb);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

extern "C" int uniql_dequant(const uint8_t* packed, const void* scales, const void* zeros, int64_t N,
                             int64_t K, int dt, void* w, void* stream) {
  if (!packed || !scales || !zeros || !w) return UNIQL_ERR_NULL;
  if (N < 0 || K < 0 || (K % kGroup)) return UNIQL_ERR_SHAPE;
  if (dt != UNIQL_F16 && dt != UNIQL_BF16) return UNIQL_ERR_DTYPE;
  int64_t nb = N * (K / 2);
  if (nb == 0) return UNIQL_OK;
  if (dt == UNIQL_F16)
    dequant_kernel<__half><<<grid_for(nb, 256), 256, 0, (cudaStream_t)stream>>>(
        packed, (const __half*)scales, (const __half*)zeros, N, K, (__half*)w);
  else
    dequant_kernel<__nv_bfloat16><<<grid_for(nb, 256), 256, 0, (cudaStream_t)stream>>>(
        packed, (const __half*)scales, (const __half*)zeros, N, K, (__nv_bfloat16*)w);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}

extern "C" int uniql_embed_rows(const uint8_t* packed, const void* scales, const void* zeros, int64_t V, int64_t K,
                                const int32_t* ids, int64_t M, int dt, void* out, int64_t ldo, int* bad_id,
                                void* stream) {
  if (!packed || !scales || !zeros || !ids || !out) return UNIQL_ERR_NULL;
  if (V < 1 || K < kGroup || (K % kGroup) || M < 0 || ldo < K) return UNIQL_ERR_SHAPE;
  if (M > 65535) return UNIQL_ERR_SHAPE;
  if (dt != UNIQL_F16 && dt != UNIQL_BF16) return UNIQL_ERR_DTYPE;
  if ((((uintptr_t)packed) & 3) || (((uintptr_t)ids) & 3) || (((uintptr_t)out) & 1) || (bad_id && (((uintptr_t)bad_id) & 3)))
    return UNIQL_ERR_ALIGN;
  if (M == 0) return UNIQL_OK;
  const int threads = 128;
  int bx = (int)((K / 8 + threads - 1) / threads);
  if (bx > 64) bx = 64;
  dim3 grid(bx, (unsigned)M);
  if (dt == UNIQL_F16)
    embed_kernel<__half><<<grid, threads, 0, (cudaStream_t)stream>>>(packed, (const __half*)scales, (const __half*)zeros,
                                                                      V, K, ids, (__half*)out, ldo, bad_id);
  else
    embed_kernel<__nv_bfloat16><<<grid, threads, 0, (cudaStream_t)stream>>>(
        packed, (const __half*)scales, (const __half*)zeros, V, K, ids, (__nv_bfloat16*)out, ldo, bad_id);
  return cudaGetLastError() == cudaSuccess ? UNIQL_OK : UNIQL_ERR_CUDA;
}
