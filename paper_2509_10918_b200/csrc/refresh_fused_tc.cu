// Destination selection and merge weights of a 64-token tile in one kernel (Sec. 4.1, Algorithm 2 and
// Sec. 4.2.1), for the refresh steps of the small-tile block: instead of a Gram kernel, a greedy kernel, a
// gather and a weights kernel - four launches of a few microseconds of work each - one CTA per tile
//   1. streams the tile's quantised tokens y and its raw tokens x (64-channel slabs, TMA ring) through two
//      Gram products on the tensor cores: S = y y^T (exact in fp32: every partial sum is a multiple of 2^-24
//      below 1) and G = x x^T, both 64 x 64 in tensor memory;
//   2. rounds S to the fixed-point S_q in shared memory and runs the greedy rounds on it in ONE warp (two
//      candidates and two cached maxima per lane: no barrier, no list; a round is a warp reduction, two row
//      reads, two ballots and a walk over the few columns whose maximum improved);
//   3. takes the logits of Sec. 4.2.1 out of G - the logit of source k and destination i is G[idx_i][k] scaled,
//      so no second contraction and no gathered copy of the destinations is needed -, softmax over the
//      destinations per source, row sums per destination in a fixed order, and writes A~^T as hi and lo planes.
// The quantised tokens come from quantise_kernel (fp64 arithmetic over 148 SMs; one CTA per tile would take
// longer over it than the kernel takes as a whole).
// Warp 0, 1: thread = token = tensor-memory lane (warp 0 runs the greedy rounds); warp 2: TMA producer;
// warp 3: MMA issuer.
#include <climits>

#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kTok = 64;            // tokens per tile this kernel is written for
constexpr int kSlab = kTok * 128;   // one 64-channel slab of 64 tokens
constexpr int kStageBytes = 2 * kSlab;  // y slab, then x slab
constexpr int kRing = 8;            // stages: 128 KB in flight per CTA (few CTAs: bytes in flight are what counts)
constexpr int kPitch = kTok + 1;    // fp32 row pitch of G and of the shares in shared memory (conflict-free both ways)

struct RBars {
  uint64_t full[kRing], empty[kRing], done;
  uint32_t tmem_base;
  int abort_flag;
  int go;  // the row warps' common decision to carry on after the contractions
};

struct RParams {
  int P, tiles_x, th, tw, d, Dloc;
  float scale_log2;  // log2(e) / (tau * sqrt(d))
  int32_t* idx;      // [tile][D_loc]
  __nv_bfloat16* w;  // A~^T planes: [tile][hi, lo][64 tokens][D_loc]
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Greedy rounds of Algorithm 2 on a 64 x 64 S_q in shared memory, by one warp.  Lane l owns candidates l and
// l + 32 (their gains) and the cached maxima m[l], m[l + 32].  Exact integer gains, ties to the lowest index,
// selected tokens excluded: the same picks as greedy_kernel.
__device__ __forceinline__ void greedy_one_warp(const int16_t* S, int Dloc, int lane, int* sel, int32_t* out) {
  const int j0 = lane, j1 = lane + 32;
  int sum0 = 0, sum1 = 0;
  for (int i = 0; i < kTok; ++i) {
    sum0 += S[i * kTok + j0];
    sum1 += S[i * kTok + j1];
  }
  // first pick: argmax of the column sums (they may be negative), lowest index on ties
  int g = sum0 >= sum1 ? sum0 : sum1, gi = sum0 >= sum1 ? j0 : j1;
  const int gmax = __reduce_max_sync(0xffffffffu, g);
  int pick = __reduce_min_sync(0xffffffffu, g == gmax ? gi : INT_MAX);
  bool sel0 = pick == j0, sel1 = pick == j1;
  if (lane == 0) {
    sel[0] = pick;
    out[0] = pick;
  }
  int m0 = S[pick * kTok + j0], m1 = S[pick * kTok + j1];
  int g0 = 0, g1 = 0;
  {
    const int16_t* mrow = S + pick * kTok;
    for (int i = 0; i < kTok; ++i) {
      const int mi = mrow[i];
      g0 += max((int)S[i * kTok + j0] - mi, 0);
      g1 += max((int)S[i * kTok + j1] - mi, 0);
    }
  }
  for (int r = 1; r < Dloc; ++r) {
    // gain (< 2^23) and 255 - index in one positive key: the largest key is the largest gain, lowest index
    const int k0 = sel0 ? -1 : (g0 << 8) | (255 - j0), k1 = sel1 ? -1 : (g1 << 8) | (255 - j1);
    pick = 255 - (__reduce_max_sync(0xffffffffu, max(k0, k1)) & 255);
    sel0 = sel0 || pick == j0;
    sel1 = sel1 || pick == j1;
    if (lane == 0) {
      sel[r] = pick;
      out[r] = pick;
    }
    const int s0 = S[pick * kTok + j0], s1 = S[pick * kTok + j1];
    unsigned b0 = __ballot_sync(0xffffffffu, s0 > m0), b1 = __ballot_sync(0xffffffffu, s1 > m1);
    // columns whose cached maximum improves: g_j += relu(S[i][j] - new) - relu(S[i][j] - old)
    while (b0) {
      const int l = __ffs(b0) - 1;
      b0 &= b0 - 1;
      const int old = __shfl_sync(0xffffffffu, m0, l), nw = __shfl_sync(0xffffffffu, s0, l);
      const int v0 = S[l * kTok + j0], v1 = S[l * kTok + j1];
      g0 += max(v0 - nw, 0) - max(v0 - old, 0);
      g1 += max(v1 - nw, 0) - max(v1 - old, 0);
    }
    while (b1) {
      const int l = __ffs(b1) - 1;
      b1 &= b1 - 1;
      const int old = __shfl_sync(0xffffffffu, m1, l), nw = __shfl_sync(0xffffffffu, s1, l);
      const int v0 = S[(l + 32) * kTok + j0], v1 = S[(l + 32) * kTok + j1];
      g0 += max(v0 - nw, 0) - max(v0 - old, 0);
      g1 += max(v1 - nw, 0) - max(v1 - old, 0);
    }
    m0 = max(m0, s0);
    m1 = max(m1, s1);
  }
}

__device__ __forceinline__ void rows_sync() { asm volatile("bar.sync 1, 64;" ::: "memory"); }  // warps 0 and 1

__global__ void __launch_bounds__(128, 1)
refresh_small_kernel(const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_x, const RParams p,
                     uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // ring, then one slab of padding: an MMA reads 128 operand rows, of which only the first 64 exist; the other 64
  // are whatever follows the slab (their accumulator rows are never read)
  uint8_t* ring = smem;
  int16_t* S = reinterpret_cast<int16_t*>(ring + kRing * kStageBytes + kSlab);  // [64][64]
  float* G = reinterpret_cast<float*>(S + kTok * kTok);                         // [64][kPitch]
  float* A = G + kTok * kPitch;                                                 // shares [D_loc][kPitch]
  float* zinv = A + kTok * kPitch;                                              // [64]
  int* sel = reinterpret_cast<int*>(zinv + kTok);                               // [64]
  RBars* bar = reinterpret_cast<RBars*>(sel + kTok);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_b = blockIdx.x, b = tile_b / p.P, tile = tile_b - b * p.P;
  const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
  const int nk = p.d / 64;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRing; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_y);
    prefetch_tmap(&tm_x);
  }
  dependency_wait();  // before tensor memory is held and before any global access
  if (threadIdx.x == 0) release_dependents();
  if (warp == 3) tmem_alloc(&bar->tmem_base, 128);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 2) {
    if (elect_one()) {
      for (int k = 0; k < nk; ++k) {
        const int s = k % kRing;
        if (k >= kRing && !mbar_wait(&bar->empty[s], ((k / kRing) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* st = ring + s * kStageBytes;
        mbar_expect_tx(&bar->full[s], kStageBytes);
        tma_load_3d(st, &tm_y, &bar->full[s], k * 64, 0, tile_b);
        tma_load_4d(st + kSlab, &tm_x, &bar->full[s], k * 64, tx * p.tw, ty * p.th, b);
      }
    }
  } else if (warp == 3) {
    if (elect_one()) {
      constexpr uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, kTok);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % kRing;
        if (!mbar_wait(&bar->full[s], (k / kRing) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ya = smem_u32(ring + s * kStageBytes), xa = ya + kSlab;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {  // 16 channels per MMA
          const uint64_t yd = smem_desc_sw128(ya + kk * 32, 16, 1024), xd = smem_desc_sw128(xa + kk * 32, 16, 1024);
          mma_ss(tmem, yd, yd, idesc, k > 0 || kk > 0);
          mma_ss(tmem + kTok, xd, xd, idesc, k > 0 || kk > 0);
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int r = threadIdx.x;  // token = tensor-memory lane (warp 0: lanes 0..31, warp 1: 32..63)
    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
    // one answer per warp: the tensor-memory loads below are warp-wide operations
    if (__all_sync(0xffffffffu, mbar_wait(&bar->done, 0, dev_status, abort_flag))) {
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < kTok; c0 += 32) {  // S_q[r][c] = rint(<y_r, y_c> * 4096), the diagonal by definition
        uint32_t v[32];
        tmem_ld32(taddr + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          S[(c0 + e) * kTok + r] = (c0 + e == r) ? (int16_t)kDiagQ : (int16_t)__float2int_rn(__uint_as_float(v[e]) * 4096.f);
      }
#pragma unroll
      for (int c0 = 0; c0 < kTok; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(taddr + kTok + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) G[r * kPitch + c0 + e] = __uint_as_float(v[e]);
      }
    }
    rows_sync();  // S_q and G are complete in shared memory - or somebody's wait ran out
    if (r == 0) bar->go = *abort_flag ? 0 : 1;  // one decision for both warps: the barriers below need all 64 threads
    rows_sync();
    if (bar->go) {
      // ---- Algorithm 2
      if (warp == 0) greedy_one_warp(S, p.Dloc, lane, sel, p.idx + (size_t)tile_b * p.Dloc);
      rows_sync();
      // ---- Sec. 4.2.1: thread = source token k; logit of destination i is G[idx_i][k] / (tau sqrt(d))
      const int Dl = p.Dloc;
      float mx = -INFINITY;
      for (int i = 0; i < Dl; ++i) mx = fmaxf(mx, G[sel[i] * kPitch + r]);
      const float neg_m = -mx * p.scale_log2;
      float sum = 0.f;
      for (int i = 0; i < Dl; ++i) sum += ex2(fmaf(G[sel[i] * kPitch + r], p.scale_log2, neg_m));
      const float inv = 1.f / sum;
      for (int i = 0; i < Dl; ++i) A[i * kPitch + r] = ex2(fmaf(G[sel[i] * kPitch + r], p.scale_log2, neg_m)) * inv;
      rows_sync();
      if (r < Dl) {  // row sum of destination r over the tile's sources, in source order
        float z = 0.f;
        for (int k = 0; k < kTok; ++k) z += A[r * kPitch + k];
        zinv[r] = z > 0.f ? 1.f / z : 0.f;  // a row sum that underflowed to 0 gives a zero row
      }
      rows_sync();
      // A~^T[k][i] = A[i][k] / Z_i as hi + lo bf16 planes; a source's D_loc weights are contiguous (D_loc % 8 == 0)
      __nv_bfloat16* hi_row = p.w + ((size_t)tile_b * 2 * kTok + r) * Dl;
      __nv_bfloat16* lo_row = hi_row + (size_t)kTok * Dl;
      for (int i0 = 0; i0 < Dl; i0 += 8) {
        __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v = A[(i0 + e) * kPitch + r] * zinv[i0 + e];
          hi[e] = __float2bfloat16_rn(v);
          lo[e] = __float2bfloat16_rn(v - __bfloat162float(hi[e]));
        }
        *reinterpret_cast<uint4*>(hi_row + i0) = *reinterpret_cast<const uint4*>(hi);
        *reinterpret_cast<uint4*>(lo_row + i0) = *reinterpret_cast<const uint4*>(lo);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 3) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

constexpr int kRefreshSmem = 1024 + kRing * kStageBytes + kSlab + kTok * kTok * 2 + 2 * kTok * kPitch * 4 + 2 * kTok * 4 + 256;
static_assert(sizeof(RBars) <= 256, "barrier block outgrew its reservation");

}  // namespace

// Shapes the one-kernel selection + weights covers: bf16 tokens, tile-local merge, tiles of 64 tokens that are one
// 4-D TMA box, destinations in whole 16-byte rows of the weight planes, whole 64-channel slabs, and no second
// (shares) matrix behind the weights.
bool refresh_fused_supported(const Geom& g) {
  if (g.f32 || g.global_merge || g.unmerge_mode != TOMA_UNMERGE_TRANSPOSE) return false;
  if (g.Nloc != kTok || g.tw > 64 || 64 % g.tw != 0 || g.th != 64 / g.tw) return false;
  if (g.Dloc < 1 || g.Dloc > kTok || g.Dloc % 8 != 0 || g.d % 64 != 0) return false;
  return true;
}

// `y`: the tile-major quantised tokens (launch_quantise).  Writes idx and the weight planes.
cudaError_t launch_refresh_fused(const Geom& g, const __nv_bfloat16* y, const void* x, int32_t* idx, void* w, uint32_t* dev_status,
                                 cudaStream_t s) {
  CUtensorMap ty, tx;
  const uint64_t ydims[3] = {(uint64_t)g.d, (uint64_t)g.Nloc, (uint64_t)g.B * g.P};
  const uint64_t ystrides[2] = {(uint64_t)g.d * 2, (uint64_t)g.Nloc * g.d * 2};
  const uint32_t ybox[3] = {64, (uint32_t)kTok, 1};
  const uint64_t xdims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t xstrides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t xbox[4] = {64, (uint32_t)g.tw, (uint32_t)g.th, 1};
  if (!encode_tmap_16bit(&ty, y, 3, ydims, ystrides, ybox) || !encode_tmap_16bit(&tx, x, 4, xdims, xstrides, xbox))
    return cudaErrorInvalidValue;
  RParams p;
  p.P = g.P; p.tiles_x = g.tiles_x; p.th = g.th; p.tw = g.tw; p.d = g.d; p.Dloc = g.Dloc;
  p.scale_log2 = g.logit_scale * 1.4426950408889634f;
  p.idx = idx;
  p.w = (__nv_bfloat16*)w;
  static std::atomic<unsigned long long> raised{0};
  cudaError_t e = raise_dynamic_smem(refresh_small_kernel, kRefreshSmem, raised);
  if (e != cudaSuccess) return e;
  e = launch_dependent(refresh_small_kernel, dim3(g.B * g.P), dim3(128), (size_t)kRefreshSmem, s, ty, tx, p, dev_status);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace toma
