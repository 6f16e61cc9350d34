// uniql_qlinear_noalloc: the decode linear layer for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a serving loop whose memory
// pool was sized at start-up and handed out completely, inside a real-time callback where an
// allocation could block on the driver, or in a sandbox that forbids it.  The regular entry points
// either take a caller workspace or let the library allocate one at first use.  This entry point does
// neither: the scratch memory of the decode kernel (arrival counters, status word, partial sums of
// tiles shared by several thread blocks) is a fixed array in the library's device image.
#include <string.h>

#include <mutex>

#include "common.cuh"

using namespace uniql;

// Lives in every GPU context that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[UNIQL_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDev = 64;
void* g_scratch_addr[kMaxDev] = {nullptr};
std::mutex g_scratch_mutex;

// Device address of the array on the current device.  The array's name is only a handle in host code;
// the address a kernel can use has to be asked for, once per device, with that device current.
int scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return UNIQL_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return UNIQL_ERR_CUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return UNIQL_OK;
}

}  // namespace

extern "C" int uniql_qlinear_noalloc(const void* x, const uint8_t* packed_w, const void* scales, const void* zeros,
                                     int M, int K, int N, int k_in, int k_out, void* y, void* stream) {
  if (!x || !packed_w || !scales || !zeros || !y) return UNIQL_ERR_NULL;
  if (M < 1 || K < kGroup || (K % kGroup) != 0 || N < 1) return UNIQL_ERR_SHAPE;
  if (k_in < 4 || k_in > K || (k_in % 4) || k_out < 4 || k_out > N || (k_out % 4)) return UNIQL_ERR_SHAPE;
  if (M > 16) return UNIQL_ERR_UNSUPPORTED;      // only the decode kernel needs (and here: has) scratch
  if ((((uintptr_t)x) & 1) || (((uintptr_t)y) & 1) || (((uintptr_t)packed_w) & 15) || (((uintptr_t)scales) & 1) ||
      (((uintptr_t)zeros) & 1))
    return UNIQL_ERR_ALIGN;
  if (cudaPeekAtLastError() != cudaSuccess) return UNIQL_ERR_CUDA;

  Params p;
  memset(&p, 0, sizeof(p));
  p.x = x; p.ldx = k_in; p.dt = UNIQL_F16; p.M = M; p.K = K; p.k_in = k_in;
  p.imap.n_fam = 1; p.imap.total = k_in; p.imap.fam[0] = Fam{0, k_in, k_in, 1}; p.imap.base[0] = 0;
  p.n_jobs = 1;
  JobDev& d = p.job[0];
  d.w = packed_w; d.scales = (const __half*)scales; d.zeros = (const __half*)zeros; d.bias = nullptr;
  d.y = y; d.ldy = k_out; d.N = N; d.k_out = k_out;
  d.omap.n_fam = 1; d.omap.total = k_out; d.omap.fam[0] = Fam{0, k_out, k_out, 1}; d.omap.base[0] = 0;
  if (!decode_supported(p)) return UNIQL_ERR_UNSUPPORTED;

  void* scratch = nullptr;
  int rc = scratch_address(&scratch);
  if (rc != UNIQL_OK) return rc;
  // The array keeps whatever the previous call left.  Counters and the status word must start at zero (they do
  // return to zero after a call that ran to its end, but not after one that gave up): the launcher clears them
  // on `stream`, after its own checks, so a call that is turned down puts nothing on the stream.
  LaunchCfg cfg{scratch, (size_t)UNIQL_NOALLOC_SCRATCH_BYTES, (cudaStream_t)stream, 1};
  return launch_decode(p, cfg);      // UNIQL_ERR_WORKSPACE when the problem needs more than the fixed array
}

// The status word of the calls above lives inside the fixed array, where uniql_workspace_status cannot see it.
extern "C" int uniql_noalloc_status(int* status) {
  if (!status) return UNIQL_ERR_NULL;
  void* scratch = nullptr;
  const int rc = scratch_address(&scratch);
  if (rc != UNIQL_OK) return rc;
  int v = 0;
  // (a blocking copy on the legacy stream: it waits for the work in flight and allocates nothing)
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&v, reinterpret_cast<unsigned char*>(scratch) + decode_status_offset(), sizeof(int),
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return UNIQL_ERR_CUDA;
  *status = v;
  return UNIQL_OK;
}
