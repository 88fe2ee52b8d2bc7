// toma_select_static: destination selection for callers that cannot supply a workspace.
//
// Who needs this: code that is handed nothing but its tensors and a stream -- an inference
// runtime's per-layer hook, a plug-in called from inside someone else's step loop -- and that must
// not allocate device memory at that point, because cudaMalloc/cudaFree synchronise the whole
// device, are forbidden while a stream is being captured, and would bypass the host framework's
// own memory pool (which may already own all free memory).  For them the scratch that toma_select
// normally takes from the caller's workspace lives in a fixed static device array inside this
// library instead.
//
// Consequences the caller has to know:
//   * The array (TOMA_STATIC_SCRATCH_BYTES) belongs to this library's device code.  With the CUDA
//     runtime's default lazy loading, a device reserves it when that code is first loaded there,
//     which is the first toma_select_static call on that device, and keeps it until the process
//     exits; with eager loading every device that initialises the library holds it from then on.
//     Either way that first call is where the reservation can fail (no free memory left on the
//     device): it then returns TOMA_ERR_CUDA, launches nothing, and leaves no sticky error behind.
//   * Problems whose scratch (quantised tokens + int16 similarity matrices) does not fit are
//     rejected with TOMA_ERR_SCRATCH_LIMIT before anything is launched.
//   * All calls on one device share the one array and it keeps whatever the previous call left.
//     Nothing in it has to start at zero: each call first writes every byte it later reads.  Two
//     calls that may overlap on the GPU (different streams, no dependency) race on it; callers
//     must order them.
//   * The first call on each device looks the array's device address up (cudaGetSymbolAddress with
//     that device current; this is what loads the code and reserves the array, see above).  Make
//     that first call outside any stream capture.
// Nothing here calls cudaMalloc, cudaFree or any allocating routine.
#include <mutex>

#include "common.cuh"

namespace toma {

// In host code `g_select_scratch` is only a handle for the symbol, not a device address; the address
// each device uses is resolved below and passed to the kernels as an ordinary pointer.
static __device__ __align__(256) unsigned char g_select_scratch[TOMA_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the static scratch on the current device (resolved once per device).
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_select_scratch);
    if (e != cudaSuccess) {
      (void)cudaGetLastError();  // the failed lookup must not surface again in the caller's next CUDA call
      return e;
    }
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace
}  // namespace toma

using namespace toma;

extern "C" toma_status toma_select_static(const toma_desc* desc, const void* x, int32_t* idx, uint32_t* dev_status,
                                          void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!x || !idx) return TOMA_ERR_NULL;
  if (((uintptr_t)x & 15) != 0) return TOMA_ERR_SHAPE;
  const size_t tiles = (size_t)g.B * g.P;
  const size_t y_bytes = align256(tiles * g.Nloc * g.d * sizeof(__nv_bfloat16));
  const size_t sq_bytes = align256(tiles * g.Nloc * g.Nloc * sizeof(int16_t));
  if (y_bytes + sq_bytes > (size_t)TOMA_STATIC_SCRATCH_BYTES) return TOMA_ERR_SCRATCH_LIMIT;
  void* base = nullptr;
  if (scratch_for_current_device(&base) != cudaSuccess) return TOMA_ERR_CUDA;
  __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(base);
  int16_t* sq = reinterpret_cast<int16_t*>(static_cast<unsigned char*>(base) + y_bytes);
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = launch_quantise(g, x, y, s);
  if (e == cudaSuccess) e = gram_tc_supported(g) ? launch_gram_tc(g, y, sq, dev_status, s) : launch_gram_ffma(g, y, sq, s);
  if (e == cudaSuccess) e = launch_greedy(g, sq, idx, s);
  return e == cudaSuccess ? TOMA_OK : TOMA_ERR_CUDA;
}
