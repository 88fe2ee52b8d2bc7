// Destination selection (Sec. 4.1, Algorithm 2): token quantisation, the
// fixed-point Gram matrix per tile (plain FFMA version) and the greedy
// facility-location argmax with exact incremental integer gains.
#include "common.cuh"
#include "tc.cuh"

namespace toma {

// ---------------------------------------------------------------------------
// Quantise: one warp per image token.  y = bf16(rint(x * 0.99*4096/|x|) * 2^-12)
// written tile-major: row (b*P + p)*N_loc + l.  fp64 arithmetic so that the CPU
// definition can be matched bit for bit.
// ---------------------------------------------------------------------------
// Eight consecutive elements as floats (16-byte aligned source).
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 f = __bfloat1622float2(h[e]);
    v[2 * e] = f.x;
    v[2 * e + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

template <typename T>
__global__ void __launch_bounds__(256) quantise_kernel(const T* __restrict__ x, __nv_bfloat16* __restrict__ y, int B,
                                                       int N, int n_all, int d, int W, int th, int tw, int tiles_x,
                                                       int P, int Nloc) {
  tc::dependency_wait();  // launched with programmatic stream serialisation
  if (threadIdx.x == 0) tc::release_dependents();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= B * N) return;
  const int b = warp / N, n = warp - b * N;
  const int yy = n / W, xx = n - yy * W;
  const int p = (yy / th) * tiles_x + xx / tw;
  const int l = (yy % th) * tw + xx % tw;
  const T* row = x + ((size_t)b * n_all + n) * d;
  __nv_bfloat16* out = y + ((size_t)(b * P + p) * Nloc + l) * d;
  // eight channels (16 or 32 contiguous bytes) per lane and trip; dim is a multiple of 8
  double ss = 0.0;
  for (int c = lane * 8; c < d; c += 256) {
    float v[8];
    load8(row + c, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss += (double)v[e] * (double)v[e];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const double scale = kCosScaleTimesOne / fmax(sqrt(ss), 1e-30);
  for (int c = lane * 8; c < d; c += 256) {  // second read of the row: an L1/L2 hit
    float v[8];
    load8(row + c, v);
    __align__(16) __nv_bfloat16 q[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) q[e] = __float2bfloat16_rn((float)rint((double)v[e] * scale) * (1.0f / 4096.0f));
    *reinterpret_cast<uint4*>(out + c) = *reinterpret_cast<const uint4*>(q);
  }
}

cudaError_t launch_quantise(const Geom& g, const void* x, __nv_bfloat16* y, cudaStream_t s) {
  const long long warps = (long long)g.B * g.N;
  const int blocks = (int)((warps * 32 + 255) / 256);
  cudaError_t e;
  if (g.f32)
    e = launch_dependent(quantise_kernel<float>, dim3(blocks), dim3(256), 0, s, (const float*)x, y, g.B, g.N, (int)g.tokens_all(), g.d, g.W, g.th,
                                                  g.tw, g.tiles_x, g.P, g.Nloc);
  else
    e = launch_dependent(quantise_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, s, (const __nv_bfloat16*)x, y, g.B, g.N, (int)g.tokens_all(),
                                                          g.d, g.W, g.th, g.tw, g.tiles_x, g.P, g.Nloc);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Gram, FFMA version: S_q[i][j] = rint(<y_i, y_j> * 4096), diag = 4014.
// 64x64 output block per CTA, 4x4 per thread, 32-channel chunks in shared memory.
// The fp32 sum is exact in any order (every partial sum is a multiple of 2^-24
// below 1), so this equals the integer definition.  Used for tile sizes the
// tensor-core version does not cover.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gram_ffma_kernel(const __nv_bfloat16* __restrict__ y,
                                                        int16_t* __restrict__ sq, int Nloc, int d) {
  __shared__ float As[32][65];
  __shared__ float Bs[32][65];
  const int tile = blockIdx.z;
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  const __nv_bfloat16* Y = y + (size_t)tile * Nloc * d;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int c0 = 0; c0 < d; c0 += 32) {
    for (int e = threadIdx.x; e < 64 * 32; e += 256) {
      const int r = e >> 5, c = e & 31;
      const bool cin = c0 + c < d;
      As[c][r] = (cin && i0 + r < Nloc) ? __bfloat162float(Y[(size_t)(i0 + r) * d + c0 + c]) : 0.f;
      Bs[c][r] = (cin && j0 + r < Nloc) ? __bfloat162float(Y[(size_t)(j0 + r) * d + c0 + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int c = 0; c < 32; ++c) {
      float a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a[u] = As[c][ty * 4 + u];
        b[u] = Bs[c][tx * 4 + u];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
    }
    __syncthreads();
  }
  int16_t* S = sq + (size_t)tile * Nloc * Nloc;
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = i0 + ty * 4 + u, j = j0 + tx * 4 + v;
      if (i < Nloc && j < Nloc)
        S[(size_t)i * Nloc + j] = (i == j) ? (int16_t)kDiagQ : (int16_t)__float2int_rn(acc[u][v] * 4096.f);
    }
}

cudaError_t launch_gram_ffma(const Geom& g, const __nv_bfloat16* y, int16_t* sq, cudaStream_t s) {
  dim3 grid((g.Nloc + 63) / 64, (g.Nloc + 63) / 64, g.B * g.P);
  gram_ffma_kernel<<<grid, 256, 0, s>>>(y, sq, g.Nloc, g.d);
  count_launch();
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Greedy (Algorithm 2), one CTA per tile, one thread per candidate token.
//
// Gains are kept incrementally and exactly: after a pick t only the columns j
// with S[t][j] > m[j] change the cached maximum, and for those
//   g_i += relu(S[i][j] - m_new[j]) - relu(S[i][j] - m_old[j]).
// All quantities are integers, so this equals recomputing
//   g_i = sum_j relu(S[i][j] - m[j])
// from scratch every round.  S is symmetric; it is always read as S[j][i] with
// i = thread index so that a warp reads consecutive int16.  Thread i also owns
// m[i] in a register.  For N_loc <= 256 the tile's S_q (<= 128 KB) is first
// copied to shared memory so that the two dependent reads of every round cost a
// shared-memory latency instead of an L2 round trip.
// Two block barriers per round: after the per-warp argmax partials are posted,
// and after the changed-column list is posted (both double buffered).
// Ties: lowest index.  Selected tokens are excluded from the argmax.
// ---------------------------------------------------------------------------
struct ArgMax {
  int g, i;
};
// Warp argmax with lowest-index ties: two hardware warp reductions (redux.sync).
__device__ __forceinline__ ArgMax warp_argmax(ArgMax v) {
  const int g = __reduce_max_sync(0xffffffffu, v.g);
  const int i = __reduce_min_sync(0xffffffffu, v.g == g ? v.i : INT_MAX);
  return ArgMax{g, i};
}
// Posts this warp's best into red[], one barrier, then every warp reduces the partials itself.
__device__ __forceinline__ ArgMax block_argmax(ArgMax v, ArgMax* red, int nwarps) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_argmax(v);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  return warp_argmax(lane < nwarps ? red[lane] : ArgMax{INT_MIN, INT_MAX});
}

// Argmax for tiles of at most 256 tokens (8 warps): gain (< 2^23) and index packed into one positive
// int, gain in the high bits and 255 - index below, so that the largest key is the largest gain with
// the lowest index; -1 never wins.  One warp reduction, one barrier, then every thread takes the
// maximum of the eight warp keys itself (two 16-byte shared loads instead of two more reductions).
__device__ __forceinline__ int block_argmax_packed(int gain, int i, bool candidate, int* keys /*[8], 16-byte aligned*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int key = __reduce_max_sync(0xffffffffu, candidate ? (gain << 8) | (255 - i) : -1);
  if (lane == 0) keys[warp] = key;
  __syncthreads();
  const int4 a = reinterpret_cast<const int4*>(keys)[0], b = reinterpret_cast<const int4*>(keys)[1];
  const int best = max(max(max(a.x, a.y), max(a.z, a.w)), max(max(b.x, b.y), max(b.z, b.w)));
  return 255 - (best & 255);
}

template <bool kSmemS>
__global__ void __launch_bounds__(1024) greedy_kernel(const int16_t* __restrict__ sq, int32_t* __restrict__ idx,
                                                      int Nloc, int Dloc) {
  extern __shared__ __align__(16) uint8_t greedy_smem[];
  // (column j, new << 16 | old & 0xffff) of columns whose cached maximum improved; cleared at the start and padded,
  // so that the entries behind a list's end are readable and name a valid column
  __shared__ int2 changed[2][kMaxNloc + 4];
  __shared__ ArgMax red[2][32];
  __shared__ __align__(16) int keys[2][8];  // warp keys of block_argmax_packed (unused slots stay -1)
  __shared__ int n_changed[2];
  const int16_t* Sg = sq + (size_t)blockIdx.x * Nloc * Nloc;
  const int16_t* S = Sg;
  if (threadIdx.x == 0) n_changed[0] = n_changed[1] = 0;
  for (int e = threadIdx.x; e < 2 * (kMaxNloc + 4); e += blockDim.x) (&changed[0][0])[e] = make_int2(0, 0);
  if (threadIdx.x < 16) keys[threadIdx.x >> 3][threadIdx.x & 7] = -1;
  tc::dependency_wait();  // launched with programmatic stream serialisation
  if (threadIdx.x == 0) tc::release_dependents();
  if (kSmemS) {
    const int n16 = Nloc * Nloc / 8;  // 16-byte packets
    const uint4* src = reinterpret_cast<const uint4*>(Sg);
    uint4* dst = reinterpret_cast<uint4*>(greedy_smem);
    for (int e = threadIdx.x; e < n16; e += blockDim.x) dst[e] = src[e];
    S = reinterpret_cast<const int16_t*>(greedy_smem);
  }
  __syncthreads();
  int32_t* out = idx + (size_t)blockIdx.x * Dloc;
  const int i = threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool live = i < Nloc;
  const int nwarps = blockDim.x >> 5;
  constexpr int kNever = INT_MIN;

  // first pick: argmax of row sums (= column sums)
  int sum = 0;
  if (live)
    for (int j = 0; j < Nloc; ++j) sum += S[(size_t)j * Nloc + i];
  ArgMax pick = block_argmax(ArgMax{live ? sum : kNever, i}, red[0], nwarps);
  bool selected = false;
  if (i == pick.i) {
    selected = true;
    out[0] = pick.i;
  }
  // cached maximum m[j] = S[t1][j]; thread i keeps m[i]; the full row is needed once for the initial gains
  int m_own = live ? S[(size_t)pick.i * Nloc + i] : 0;
  int gain = 0;
  if (live) {
    const int16_t* mrow = S + (size_t)pick.i * Nloc;
    for (int j = 0; j < Nloc; ++j) gain += max((int)S[(size_t)j * Nloc + i] - (int)mrow[j], 0);
  }

  for (int r = 1; r < Dloc; ++r) {
    const int pb = r & 1;
    if (kSmemS) pick.i = block_argmax_packed(gain, i, live && !selected, keys[pb]);  // N_loc <= 256
    else pick = block_argmax(ArgMax{(live && !selected) ? gain : kNever, i}, red[pb], nwarps);
    if (i == pick.i) {
      selected = true;
      out[r] = pick.i;
    }
    const int s_new = live ? (int)S[(size_t)pick.i * Nloc + i] : 0;
    const bool ch = live && s_new > m_own;
    const unsigned mask = __ballot_sync(0xffffffffu, ch);
    // columns whose cached maximum improves, compacted into a list (one shared-memory atomic per warp)
    if (mask) {
      int base = 0;
      if (lane == 0) base = atomicAdd(&n_changed[pb], __popc(mask));
      base = __shfl_sync(0xffffffffu, base, 0);
      if (ch) {
        changed[pb][base + __popc(mask & ((1u << lane) - 1u))] =
            make_int2(i, (int)(((unsigned)s_new << 16) | ((unsigned)m_own & 0xFFFFu)));
        m_own = s_new;
      }
    }
    __syncthreads();
    const int n = n_changed[pb];
    if (threadIdx.x == 0) n_changed[pb ^ 1] = 0;  // last read one full round ago
    if (live) {
      // four entries at a time so that the dependent shared-memory reads overlap
      int e = 0;
      for (; e + 4 <= n; e += 4) {
        int2 c[4];
        int sv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) c[u] = changed[pb][e + u];
#pragma unroll
        for (int u = 0; u < 4; ++u) sv[u] = S[(size_t)c[u].x * Nloc + i];
#pragma unroll
        for (int u = 0; u < 4; ++u) gain += max(sv[u] - (c[u].y >> 16), 0) - max(sv[u] - (int)(short)(c[u].y & 0xFFFF), 0);
      }
      if (e < n) {  // up to three left: fetched together whether they exist or not, counted only if they do
        int2 c[3];
        int sv[3];
#pragma unroll
        for (int u = 0; u < 3; ++u) c[u] = changed[pb][e + u];
#pragma unroll
        for (int u = 0; u < 3; ++u) sv[u] = S[(size_t)c[u].x * Nloc + i];
#pragma unroll
        for (int u = 0; u < 3; ++u)
          gain += (e + u < n) ? max(sv[u] - (c[u].y >> 16), 0) - max(sv[u] - (int)(short)(c[u].y & 0xFFFF), 0) : 0;
      }
    }
  }
}

cudaError_t launch_greedy(const Geom& g, const int16_t* sq, int32_t* idx, cudaStream_t s) {
  const int threads = ((g.Nloc + 31) / 32) * 32;
  const size_t s_bytes = (size_t)g.Nloc * g.Nloc * 2;
  const bool smem_s = g.Nloc <= 256 && (g.Nloc * g.Nloc) % 8 == 0;
  cudaError_t e;
  if (smem_s) {
    static std::atomic<unsigned long long> smem_raised{0};
    e = raise_dynamic_smem(greedy_kernel<true>, 256 * 256 * 2, smem_raised);
    if (e != cudaSuccess) return e;
    e = launch_dependent(greedy_kernel<true>, dim3(g.B * g.P), dim3(threads), s_bytes, s, sq, idx, g.Nloc, g.Dloc);
  } else {
    e = launch_dependent(greedy_kernel<false>, dim3(g.B * g.P), dim3(threads), 0, s, sq, idx, g.Nloc, g.Dloc);
  }
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace toma
