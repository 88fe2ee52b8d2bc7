// Destination selection (Sec. 4.1, Algorithm 2): token quantisation, the
// fixed-point Gram matrix per tile (plain FFMA version) and the greedy
// facility-location argmax with exact incremental integer gains.
#include "common.cuh"

namespace toma {

// ---------------------------------------------------------------------------
// Quantise: one warp per image token.  y = bf16(rint(x * 0.99*4096/|x|) * 2^-12)
// written tile-major: row (b*P + p)*N_loc + l.  fp64 arithmetic so that the CPU
// definition can be matched bit for bit.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) quantise_kernel(const T* __restrict__ x, __nv_bfloat16* __restrict__ y, int B,
                                                       int N, int n_all, int d, int W, int th, int tw, int tiles_x,
                                                       int P, int Nloc) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= B * N) return;
  const int b = warp / N, n = warp - b * N;
  const int yy = n / W, xx = n - yy * W;
  const int p = (yy / th) * tiles_x + xx / tw;
  const int l = (yy % th) * tw + xx % tw;
  const T* row = x + ((size_t)b * n_all + n) * d;
  __nv_bfloat16* out = y + ((size_t)(b * P + p) * Nloc + l) * d;
  double ss = 0.0;
  for (int c = lane; c < d; c += 32) {
    const double v = (double)to_f32(row[c]);
    ss += v * v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const double scale = kCosScaleTimesOne / fmax(sqrt(ss), 1e-30);
  for (int c = lane; c < d; c += 32) {
    const double k = rint((double)to_f32(row[c]) * scale);
    out[c] = __float2bfloat16_rn((float)k * (1.0f / 4096.0f));
  }
}

cudaError_t launch_quantise(const Geom& g, const void* x, __nv_bfloat16* y, cudaStream_t s) {
  const long long warps = (long long)g.B * g.N;
  const int blocks = (int)((warps * 32 + 255) / 256);
  if (g.f32)
    quantise_kernel<float><<<blocks, 256, 0, s>>>((const float*)x, y, g.B, g.N, (int)g.tokens_all(), g.d, g.W, g.th,
                                                  g.tw, g.tiles_x, g.P, g.Nloc);
  else
    quantise_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((const __nv_bfloat16*)x, y, g.B, g.N, (int)g.tokens_all(),
                                                          g.d, g.W, g.th, g.tw, g.tiles_x, g.P, g.Nloc);
  count_launch();
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Gram, FFMA version: S_q[i][j] = rint(<y_i, y_j> * 4096), diag = 4014.
// 64x64 output block per CTA, 4x4 per thread, 32-channel chunks in shared memory.
// The fp32 sum is exact in any order (every partial sum is a multiple of 2^-24
// below 1), so this equals the integer definition.
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
      if (i < Nloc && j < Nloc) S[(size_t)i * Nloc + j] = (i == j) ? (int16_t)kDiagQ : (int16_t)__float2int_rn(acc[u][v] * 4096.f);
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
// i = thread index so that a warp reads consecutive int16.
// Ties: lowest index.  Selected tokens are excluded from the argmax.
// ---------------------------------------------------------------------------
struct ArgMax {
  int g, i;
};
__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b) {
  return (b.g > a.g || (b.g == a.g && b.i < a.i)) ? b : a;
}
__device__ __forceinline__ ArgMax block_argmax(ArgMax v, ArgMax* red, int nwarps) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ArgMax other{__shfl_xor_sync(0xffffffffu, v.g, o), __shfl_xor_sync(0xffffffffu, v.i, o)};
    v = better(v, other);
  }
  if (lane == 0) red[warp] = v;
  __syncthreads();
  ArgMax r = red[lane < nwarps ? lane : 0];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ArgMax other{__shfl_xor_sync(0xffffffffu, r.g, o), __shfl_xor_sync(0xffffffffu, r.i, o)};
    r = better(r, other);
  }
  __syncthreads();  // red[] may be rewritten by the next call
  return r;
}

__global__ void __launch_bounds__(1024) greedy_kernel(const int16_t* __restrict__ sq, int32_t* __restrict__ idx,
                                                      int Nloc, int Dloc) {
  __shared__ int m[kMaxNloc];
  __shared__ int ch_j[kMaxNloc];
  __shared__ int ch_old[kMaxNloc];
  __shared__ int ch_new[kMaxNloc];
  __shared__ ArgMax red[32];
  __shared__ int n_changed;
  const int16_t* S = sq + (size_t)blockIdx.x * Nloc * Nloc;
  int32_t* out = idx + (size_t)blockIdx.x * Dloc;
  const int i = threadIdx.x;
  const bool live = i < Nloc;
  const int nwarps = blockDim.x >> 5;
  constexpr int kNever = INT_MIN;

  // first pick: argmax of row sums (= column sums)
  int sum = 0;
  if (live)
    for (int j = 0; j < Nloc; ++j) sum += S[(size_t)j * Nloc + i];
  ArgMax pick = block_argmax(ArgMax{live ? sum : kNever, i}, red, nwarps);
  bool selected = false;
  if (i == pick.i) {
    selected = true;
    out[0] = pick.i;
  }
  if (live) m[i] = S[(size_t)pick.i * Nloc + i];
  __syncthreads();
  int gain = 0;
  if (live)
    for (int j = 0; j < Nloc; ++j) gain += max((int)S[(size_t)j * Nloc + i] - m[j], 0);

  for (int r = 1; r < Dloc; ++r) {
    if (threadIdx.x == 0) n_changed = 0;
    pick = block_argmax(ArgMax{(live && !selected) ? gain : kNever, i}, red, nwarps);
    if (i == pick.i) {
      selected = true;
      out[r] = pick.i;
    }
    if (live) {
      const int s_new = S[(size_t)pick.i * Nloc + i];
      const int s_old = m[i];
      if (s_new > s_old) {
        const int slot = atomicAdd(&n_changed, 1);
        ch_j[slot] = i;
        ch_old[slot] = s_old;
        ch_new[slot] = s_new;
        m[i] = s_new;
      }
    }
    __syncthreads();
    if (live) {
      const int n = n_changed;
      for (int e = 0; e < n; ++e) {
        const int s = S[(size_t)ch_j[e] * Nloc + i];
        gain += max(s - ch_new[e], 0) - max(s - ch_old[e], 0);
      }
    }
    __syncthreads();
  }
}

cudaError_t launch_greedy(const Geom& g, const int16_t* sq, int32_t* idx, cudaStream_t s) {
  const int threads = ((g.Nloc + 31) / 32) * 32;
  greedy_kernel<<<g.B * g.P, threads, 0, s>>>(sq, idx, g.Nloc, g.Dloc);
  count_launch();
  return cudaGetLastError();
}

}  // namespace toma
