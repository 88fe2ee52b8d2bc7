// Shared declarations of the ToMA sm_100a library: derived problem geometry,
// launch prototypes between translation units, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/toma.h"

namespace toma {

// Fixed-point cosine similarity constants (see toma_select in toma.h).
constexpr double kCosScaleTimesOne = 0.99 * 4096.0;  // token length 0.99 in units of 2^-12
constexpr int kDiagQ = 4014;                          // rint(0.99^2 * 4096)
constexpr int kMaxNloc = 1024;
constexpr int kMaxDim = 4096;

// Geometry derived from a validated descriptor.
struct Geom {
  int B, H, W, d, th, tw, tiles_x, P, N, Nloc, Dloc, D, n_extra, Lm;  // Lm = D + n_extra
  int heads, dh;
  bool f32;
  bool global_merge;  // weights / merge / unmerge over the whole image (selection stays per tile)
  int unmerge_mode;   // TOMA_UNMERGE_*: a non-zero mode keeps a second matrix behind A~^T in the weight buffer
  float logit_scale;  // 1 / (tau * sqrt(d))
  long long tokens_all() const { return (long long)N + n_extra; }
};

toma_status make_geom(const toma_desc* desc, Geom* g);

// Workspace carve-up (all offsets 256-byte aligned).
struct WsLayout {
  size_t y_off, sq_off, logits_off, wts_off, gidx_off, xm_off, att_off, att_ws_off, proj_off, total;
};
WsLayout ws_layout(const Geom& g);
// Geometry the weights, the merge and the unmerge work in: g itself, or, with global merge, the image as
// one region (P = 1, N_loc = N, D_loc = D).
Geom merge_geom(const Geom& g);

// Process-wide count of kernel launches (reported by toma_launch_counter()).
extern std::atomic<unsigned long long> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// Test-only overrides of launch heuristics (set through toma_test_set_tuning; the product path never
// writes them): attention work plan (-1 = heuristic, 0 = whole units, 1 = even cut), persistent CTA
// count of the attention kernel (0 = heuristic), tile form of the projection kernel (0 = heuristic), 1 = toma_block
// takes the three-kernel path even where the fused reuse-step kernel applies, and the separate selection and
// weights kernels where the one-kernel refresh of small tiles applies.
extern std::atomic<int> g_tune_attention_split, g_tune_attention_ctas, g_tune_linear_tile, g_tune_block_unfused;

// Number of SMs of the current device (cached per device).
int sm_count();

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device attribute: `done` holds one bit per
// device ordinal for which this kernel's limit has been raised (ordinals >= 64 are set every time).
template <typename Kernel>
cudaError_t raise_dynamic_smem(Kernel kernel, int bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  if (dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
  return cudaSuccess;
}

// ---- launchers (each returns cudaGetLastError() of its launches) ----
cudaError_t launch_quantise(const Geom& g, const void* x, __nv_bfloat16* y, cudaStream_t s);
cudaError_t launch_gram_ffma(const Geom& g, const __nv_bfloat16* y, int16_t* sq, cudaStream_t s);
bool gram_tc_supported(const Geom& g);
cudaError_t launch_gram_tc(const Geom& g, const __nv_bfloat16* y, int16_t* sq, uint32_t* dev_status, cudaStream_t s);
cudaError_t launch_greedy(const Geom& g, const int16_t* sq, int32_t* idx, cudaStream_t s);
// `wu`: where the un-normalised shares A^T go in the weight buffer's layout, or nullptr.
cudaError_t launch_weights_simt(const Geom& g, const void* x, const int32_t* idx, void* w, void* wu, float* logits,
                                cudaStream_t s);
cudaError_t launch_merge_simt(const Geom& g, const void* w, const void* x, void* xm, cudaStream_t s);
cudaError_t launch_unmerge_simt(const Geom& g, const void* w, const void* y, void* out, cudaStream_t s);
cudaError_t launch_attention_simt(int B, int L, int heads, int dh, bool f32, const void* q, const void* k,
                                  const void* v, void* o, cudaStream_t s);
bool weights_tc_supported(const Geom& g);
size_t weights_tc_scratch_bytes(const Geom& g);
cudaError_t launch_weights_tc(const Geom& g, const void* x, const int32_t* idx, void* w, void* wu, float* shares,
                              void* scratch, uint32_t* dev_status, cudaStream_t s);
bool linear_tc_supported(const Geom& g);
// `zero` / `zero_bytes` (multiple of 4, may be 0): a region the kernel clears on the side.
cudaError_t launch_merge_tc(const Geom& g, const void* w, const void* x, void* xm, void* zero, size_t zero_bytes,
                            uint32_t* dev_status, cudaStream_t s);
cudaError_t launch_unmerge_tc(const Geom& g, const void* w, const void* y, void* out, uint32_t* dev_status,
                              cudaStream_t s);
cudaError_t launch_copy_extra(const Geom& g, const void* src, void* dst, bool merging, cudaStream_t s);
// Scratch of the tensor-core attention (tickets and partial results of split work units).
size_t attention_tc_workspace_bytes(int B, int L, int heads, int dh);
// The scratch starts with the tickets (attention_tc_ticket_bytes()), which must be zero when the
// kernel starts: the launcher clears them unless `tickets_clean` says an earlier kernel on the
// stream already did.
size_t attention_tc_ticket_bytes(int B, int L, int heads);
// The work plan of a launch (see toma_attention_plan); returns the CTA count, 0 if the shape is too large.
int attention_tc_plan(int B, int L, int heads, int info[4], int* bounds, int* owner_first, int* owner_last, int capacity);
cudaError_t launch_attention_tc(int B, int L, int heads, int dh, const void* q, const void* k, const void* v, void* o,
                                void* ws, bool tickets_clean, uint32_t* dev_status, cudaStream_t s);
// The reuse step (merge, attention over the merged tokens, unmerge) as one kernel, for the shapes it is written for.
bool block_fused_supported(const Geom& g);
// ... and this device holds its launch (host-side occupancy query, cached per device).
bool block_fused_launchable(const Geom& g);
// Merge weights out of the raw Gram matrix G = X X^T of every tile (computed on the SMs that idle during the greedy
// rounds): launch_gram_raw goes directly behind launch_greedy, launch_weights_gram behind that.
bool weights_gram_supported(const Geom& g);
cudaError_t launch_gram_raw(const Geom& g, const void* x, float* G, uint32_t* dev_status, cudaStream_t s);
cudaError_t launch_weights_gram(const Geom& g, const float* G, const int32_t* idx, void* w, uint32_t* dev_status, cudaStream_t s);
// Selection and merge weights of 64-token tiles in one kernel (after launch_quantise), for the shapes it is written for.
bool refresh_fused_supported(const Geom& g);
cudaError_t launch_refresh_fused(const Geom& g, const __nv_bfloat16* y, const void* x, int32_t* idx, void* w, uint32_t* dev_status,
                                 cudaStream_t s);
cudaError_t launch_block_fused(const Geom& g, const void* w, const void* x, void* out, uint32_t* dev_status, cudaStream_t s);
// Image-level destination ids [batch][D] (tile-major, pick order) from the tile-local picks.
cudaError_t launch_global_idx(const Geom& g, const int32_t* idx, int32_t* gidx, cudaStream_t s);
// Projection c = a w (a [M][K], w [K][N], c [M][N], row-major): tensor-core form for bf16 (up to three
// weight / output pairs sharing a), FFMA form otherwise.
// `act`: kActNone, or kActGelu to apply the exact (erf) GELU to the fp32 result before it is stored.
constexpr int kActNone = 0, kActGelu = 1;
bool linear_tc_shape_ok(int M, int N, int K);
cudaError_t launch_linear_tc(int M, int N, int K, const void* a, const void* const* w, void* const* c, int n_mats, int act,
                             uint32_t* dev_status, cudaStream_t s);
cudaError_t launch_linear_simt(int M, int N, int K, bool f32, const void* a, const void* w, void* c, int act, cudaStream_t s);
cudaError_t launch_weights_export(const Geom& g, const void* w, float* dense, cudaStream_t s);
cudaError_t launch_weights_import(const Geom& g, const float* dense, void* w, cudaStream_t s);

// ---- device helpers ----
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ void from_f32(float& o, float v) { o = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16& o, float v) { o = __float2bfloat16_rn(v); }
__device__ __forceinline__ void from_f32(__half& o, float v) { o = __float2half_rn(v); }

// GELU(v) = v * Phi(v), Phi the standard normal distribution function.
__device__ __forceinline__ float gelu(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752f)); }

// Global row of image token (tile p, local slot l) inside one batch item.
__device__ __forceinline__ int tile_token(int p, int l, int tiles_x, int th, int tw, int W) {
  const int ty = p / tiles_x, tx = p - ty * tiles_x;
  const int ly = l / tw, lx = l - ly * tw;
  return (ty * th + ly) * W + tx * tw + lx;
}

}  // namespace toma
