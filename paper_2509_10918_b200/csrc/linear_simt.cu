// FFMA versions of the merge-weight logits, the column softmax / row
// normalisation (Sec. 4.2.1), the merge X_m = A~ X and the unmerge A~^T X'
// (Sec. 4.2.2).  They serve the fp32 mode (whose 1e-4 tolerance rules out
// reduced-precision tensor-core inputs) and every shape the tensor-core kernels do not
// cover.
#include "common.cuh"

namespace toma {

// C[m][n] = sum_k A(m,k) B(k,n) for one batch entry (blockIdx.z); 64x64x16 tiles,
// 256 threads, 4x4 outputs per thread.  `Op` supplies the element accessors.
template <class Op, typename AccT>
__global__ void __launch_bounds__(256) simt_gemm_kernel(Op op) {
  __shared__ float As[16][65];
  __shared__ float Bs[16][65];
  const int batch = blockIdx.z;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  AccT acc[4][4] = {};
  for (int k0 = 0; k0 < op.K; k0 += 16) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      int r, c;
      if (Op::a_k_contig) { r = e >> 4; c = e & 15; } else { r = e & 63; c = e >> 6; }
      As[c][r] = (m0 + r < op.M && k0 + c < op.K) ? op.a(batch, m0 + r, k0 + c) : 0.f;
      if (Op::b_k_contig) { r = e >> 4; c = e & 15; } else { r = e & 63; c = e >> 6; }
      Bs[c][r] = (n0 + r < op.N && k0 + c < op.K) ? op.b(batch, k0 + c, n0 + r) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a[u] = As[c][ty * 4 + u];
        b[u] = Bs[c][tx * 4 + u];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] += (AccT)a[u] * (AccT)b[v];
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int m = m0 + ty * 4 + u, n = n0 + tx * 4 + v;
      if (m < op.M && n < op.N) op.store(batch, m, n, acc[u][v]);
    }
}

struct TileMap {
  int P, tiles_x, th, tw, W, Nloc, Dloc, d, n_all, Lm;
  __device__ __forceinline__ size_t x_row(int batch, int l) const {  // row of X for tile-local slot l
    const int b = batch / P, p = batch - b * P;
    return (size_t)b * n_all + tile_token(p, l, tiles_x, th, tw, W);
  }
  __device__ __forceinline__ size_t m_row(int batch, int i) const {  // row of the merged tensor
    const int b = batch / P, p = batch - b * P;
    return (size_t)b * Lm + (size_t)p * Dloc + i;
  }
};

// Stored weights A~^T of one tile: fp32 mode keeps one fp32 plane [N_loc][D_loc]; bf16 mode keeps
// the value split into two bf16 planes, hi = bf16(v) and lo = bf16(v - hi), hi plane first, so that
// the tensor-core kernels can feed both planes as bf16 operands and still carry ~16 mantissa bits.
__device__ __forceinline__ float w_load(const float* w, int batch, size_t off, size_t plane) {
  return w[(size_t)batch * plane + off];
}
__device__ __forceinline__ float w_load(const __nv_bfloat16* w, int batch, size_t off, size_t plane) {
  const __nv_bfloat16* t = w + (size_t)batch * 2 * plane;
  return __bfloat162float(t[off]) + __bfloat162float(t[plane + off]);
}
__device__ __forceinline__ void w_store(float* w, int batch, size_t off, size_t plane, float v) {
  w[(size_t)batch * plane + off] = v;
}
__device__ __forceinline__ void w_store(__nv_bfloat16* w, int batch, size_t off, size_t plane, float v) {
  __nv_bfloat16* t = w + (size_t)batch * 2 * plane;
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  t[off] = hi;
  t[plane + off] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

static TileMap make_map(const Geom& g) {
  return TileMap{g.P, g.tiles_x, g.th, g.tw, g.W, g.Nloc, g.Dloc, g.d, (int)g.tokens_all(), g.Lm};
}

// logits[batch][i][k] = <X[idx_i], X_k> * scale
template <typename T>
struct LogitsOp {
  static constexpr bool a_k_contig = true, b_k_contig = true;
  int M, N, K;
  TileMap tm;
  const T* x;
  const int32_t* idx;
  float* logits;
  float scale;
  __device__ __forceinline__ float a(int batch, int i, int c) const {
    return to_f32(x[tm.x_row(batch, idx[(size_t)batch * tm.Dloc + i]) * tm.d + c]);
  }
  __device__ __forceinline__ float b(int batch, int c, int k) const { return to_f32(x[tm.x_row(batch, k) * tm.d + c]); }
  template <typename AccT>
  __device__ __forceinline__ void store(int batch, int i, int k, AccT v) const {
    logits[((size_t)batch * tm.Dloc + i) * tm.Nloc + k] = (float)(v * (AccT)scale);
  }
};

// xm[m_row(i)][c] = sum_k w[batch][k][i] x[x_row(k)][c]
template <typename T, typename WT>
struct MergeOp {
  static constexpr bool a_k_contig = false, b_k_contig = false;
  int M, N, K;
  TileMap tm;
  const WT* w;
  const T* x;
  T* xm;
  __device__ __forceinline__ float a(int batch, int i, int k) const {
    return w_load(w, batch, (size_t)k * tm.Dloc + i, (size_t)tm.Nloc * tm.Dloc);
  }
  __device__ __forceinline__ float b(int batch, int k, int c) const { return to_f32(x[tm.x_row(batch, k) * tm.d + c]); }
  __device__ __forceinline__ void store(int batch, int i, int c, float v) const {
    from_f32(xm[tm.m_row(batch, i) * tm.d + c], v);
  }
};

// out[x_row(k)][c] = sum_i w[batch][k][i] y[m_row(i)][c]
template <typename T, typename WT>
struct UnmergeOp {
  static constexpr bool a_k_contig = true, b_k_contig = false;
  int M, N, K;
  TileMap tm;
  const WT* w;
  const T* y;
  T* out;
  __device__ __forceinline__ float a(int batch, int k, int i) const {
    return w_load(w, batch, (size_t)k * tm.Dloc + i, (size_t)tm.Nloc * tm.Dloc);
  }
  __device__ __forceinline__ float b(int batch, int i, int c) const { return to_f32(y[tm.m_row(batch, i) * tm.d + c]); }
  __device__ __forceinline__ void store(int batch, int k, int c, float v) const {
    from_f32(out[tm.x_row(batch, k) * tm.d + c], v);
  }
};

template <class Op, typename AccT>
static void run_gemm(const Op& op, int batches, cudaStream_t s) {
  dim3 grid((op.N + 63) / 64, (op.M + 63) / 64, batches);
  simt_gemm_kernel<Op, AccT><<<grid, 256, 0, s>>>(op);
  count_launch();
}

// Softmax over the destination axis for every source token (a token's shares sum to 1).
// One thread per (tile, source k); logits[batch][i][k] is overwritten with A_ik.
__global__ void __launch_bounds__(128) softmax_dest_kernel(float* __restrict__ logits, int Nloc, int Dloc) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= Nloc) return;
  float* L = logits + (size_t)blockIdx.y * Dloc * Nloc + k;
  float mx = -INFINITY;
  for (int i = 0; i < Dloc; ++i) mx = fmaxf(mx, L[(size_t)i * Nloc]);
  float sum = 0.f;
  for (int i = 0; i < Dloc; ++i) {
    const float e = expf(L[(size_t)i * Nloc] - mx);
    L[(size_t)i * Nloc] = e;
    sum += e;
  }
  const float inv = 1.f / sum;
  for (int i = 0; i < Dloc; ++i) L[(size_t)i * Nloc] *= inv;
}

// Row normalisation: one warp per (tile, destination i); writes A~^T[k][i] = A_ik / sum_k' A_ik'
// and, when wu is given, the shares themselves, A^T[k][i] = A_ik, in the same layout.
template <typename WT>
__global__ void __launch_bounds__(256) rownorm_kernel(const float* __restrict__ A, WT* __restrict__ w, WT* __restrict__ wu,
                                                      int Nloc, int Dloc, int rows_total) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows_total) return;
  const int batch = row / Dloc, i = row - batch * Dloc;
  const float* a = A + (size_t)row * Nloc;
  float z = 0.f;
  for (int k = lane; k < Nloc; k += 32) z += a[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  const float inv = z > 0.f ? 1.f / z : 0.f;
  const size_t plane = (size_t)Nloc * Dloc;
  for (int k = lane; k < Nloc; k += 32) w_store(w, batch, (size_t)k * Dloc + i, plane, a[k] * inv);
  if (wu)
    for (int k = lane; k < Nloc; k += 32) w_store(wu, batch, (size_t)k * Dloc + i, plane, a[k]);
}

cudaError_t launch_weights_simt(const Geom& g, const void* x, const int32_t* idx, void* w, void* wu, float* logits,
                                cudaStream_t s) {
  const int batches = g.B * g.P;
  if (g.f32) {
    LogitsOp<float> op{g.Dloc, g.Nloc, g.d, make_map(g), (const float*)x, idx, logits, g.logit_scale};
    run_gemm<LogitsOp<float>, double>(op, batches, s);
  } else {
    LogitsOp<__nv_bfloat16> op{g.Dloc, g.Nloc, g.d, make_map(g), (const __nv_bfloat16*)x, idx, logits, g.logit_scale};
    run_gemm<LogitsOp<__nv_bfloat16>, float>(op, batches, s);
  }
  softmax_dest_kernel<<<dim3((g.Nloc + 127) / 128, batches), 128, 0, s>>>(logits, g.Nloc, g.Dloc);
  count_launch();
  const int rows = batches * g.Dloc;
  const int blocks = (rows * 32 + 255) / 256;
  if (g.f32)
    rownorm_kernel<float><<<blocks, 256, 0, s>>>(logits, (float*)w, (float*)wu, g.Nloc, g.Dloc, rows);
  else
    rownorm_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(logits, (__nv_bfloat16*)w, (__nv_bfloat16*)wu, g.Nloc, g.Dloc, rows);
  count_launch();
  return cudaGetLastError();
}

// Copy of the un-merged trailing tokens (rows [src_row0, src_row0 + n_extra) of every batch item).
template <typename T>
__global__ void copy_rows_kernel(const T* __restrict__ src, T* __restrict__ dst, int n_extra, int d, size_t src_stride,
                                 size_t dst_stride, size_t src_row0, size_t dst_row0) {
  const size_t per = (size_t)n_extra * d;
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= per) return;
  const int b = blockIdx.y;
  dst[(size_t)b * dst_stride + dst_row0 * d + e] = src[(size_t)b * src_stride + src_row0 * d + e];
}

template <typename T>
static void copy_extra(const Geom& g, const T* src, T* dst, bool merging, cudaStream_t s) {
  if (g.n_extra == 0) return;
  const size_t per = (size_t)g.n_extra * g.d;
  const size_t full = (size_t)g.tokens_all() * g.d, mrg = (size_t)g.Lm * g.d;
  dim3 grid((unsigned)((per + 255) / 256), g.B);
  if (merging)
    copy_rows_kernel<T><<<grid, 256, 0, s>>>(src, dst, g.n_extra, g.d, full, mrg, (size_t)g.N, (size_t)g.D);
  else
    copy_rows_kernel<T><<<grid, 256, 0, s>>>(src, dst, g.n_extra, g.d, mrg, full, (size_t)g.D, (size_t)g.N);
  count_launch();
}

cudaError_t launch_copy_extra(const Geom& g, const void* src, void* dst, bool merging, cudaStream_t s) {
  if (g.f32) copy_extra<float>(g, (const float*)src, (float*)dst, merging, s);
  else copy_extra<__nv_bfloat16>(g, (const __nv_bfloat16*)src, (__nv_bfloat16*)dst, merging, s);
  return cudaGetLastError();
}

cudaError_t launch_merge_simt(const Geom& g, const void* w, const void* x, void* xm, cudaStream_t s) {
  const int batches = g.B * g.P;
  if (g.f32) {
    MergeOp<float, float> op{g.Dloc, g.d, g.Nloc, make_map(g), (const float*)w, (const float*)x, (float*)xm};
    run_gemm<MergeOp<float, float>, float>(op, batches, s);
    copy_extra<float>(g, (const float*)x, (float*)xm, true, s);
  } else {
    MergeOp<__nv_bfloat16, __nv_bfloat16> op{g.Dloc, g.d, g.Nloc, make_map(g), (const __nv_bfloat16*)w, (const __nv_bfloat16*)x,
                                      (__nv_bfloat16*)xm};
    run_gemm<MergeOp<__nv_bfloat16, __nv_bfloat16>, float>(op, batches, s);
    copy_extra<__nv_bfloat16>(g, (const __nv_bfloat16*)x, (__nv_bfloat16*)xm, true, s);
  }
  return cudaGetLastError();
}

cudaError_t launch_unmerge_simt(const Geom& g, const void* w, const void* y, void* out, cudaStream_t s) {
  const int batches = g.B * g.P;
  if (g.f32) {
    UnmergeOp<float, float> op{g.Nloc, g.d, g.Dloc, make_map(g), (const float*)w, (const float*)y, (float*)out};
    run_gemm<UnmergeOp<float, float>, float>(op, batches, s);
    copy_extra<float>(g, (const float*)y, (float*)out, false, s);
  } else {
    UnmergeOp<__nv_bfloat16, __nv_bfloat16> op{g.Nloc, g.d, g.Dloc, make_map(g), (const __nv_bfloat16*)w, (const __nv_bfloat16*)y,
                                        (__nv_bfloat16*)out};
    run_gemm<UnmergeOp<__nv_bfloat16, __nv_bfloat16>, float>(op, batches, s);
    copy_extra<__nv_bfloat16>(g, (const __nv_bfloat16*)y, (__nv_bfloat16*)out, false, s);
  }
  return cudaGetLastError();
}

// c[m][n] = sum_k a[m][k] w[k][n] (plain projection; fp32 mode and shapes the tensor-core kernel does not take).
template <typename T>
struct LinearOp {
  static constexpr bool a_k_contig = true, b_k_contig = false;
  int M, N, K;
  const T* a_;
  const T* w_;
  T* c_;
  int act;
  __device__ __forceinline__ float a(int, int m, int k) const { return to_f32(a_[(size_t)m * K + k]); }
  __device__ __forceinline__ float b(int, int k, int n) const { return to_f32(w_[(size_t)k * N + n]); }
  template <typename AccT>
  __device__ __forceinline__ void store(int, int m, int n, AccT v) const {
    const float f = (float)v;
    from_f32(c_[(size_t)m * N + n], act == kActGelu ? gelu(f) : f);
  }
};

cudaError_t launch_linear_simt(int M, int N, int K, bool f32, const void* a, const void* w, void* c, int act, cudaStream_t s) {
  if (f32) {
    LinearOp<float> op{M, N, K, (const float*)a, (const float*)w, (float*)c, act};
    run_gemm<LinearOp<float>, float>(op, 1, s);
  } else {
    LinearOp<__nv_bfloat16> op{M, N, K, (const __nv_bfloat16*)a, (const __nv_bfloat16*)w, (__nv_bfloat16*)c, act};
    run_gemm<LinearOp<__nv_bfloat16>, float>(op, 1, s);
  }
  return cudaGetLastError();
}

// gidx[b][p * D_loc + k] = image token of tile p's k-th pick.
__global__ void global_idx_kernel(const int32_t* __restrict__ idx, int32_t* __restrict__ gidx, int P, int Dloc, int tiles_x,
                                  int th, int tw, int W, int total) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int p = (e / Dloc) % P;
  gidx[e] = tile_token(p, idx[e], tiles_x, th, tw, W);
}

cudaError_t launch_global_idx(const Geom& g, const int32_t* idx, int32_t* gidx, cudaStream_t s) {
  const int total = g.B * g.D;
  global_idx_kernel<<<(total + 255) / 256, 256, 0, s>>>(idx, gidx, g.P, g.Dloc, g.tiles_x, g.th, g.tw, g.W, total);
  count_launch();
  return cudaGetLastError();
}

// Dense fp32 A~ [batch][P][D_loc][N_loc]  <->  stored A~^T [batch][P][N_loc][D_loc].
template <typename WT, bool kExport>
__global__ void weights_convert_kernel(WT* __restrict__ w, float* __restrict__ dense, int Nloc, int Dloc, size_t total) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const size_t per = (size_t)Nloc * Dloc;
  const size_t batch = e / per, r = e - batch * per;
  const int k = (int)(r / Dloc), i = (int)(r - (size_t)k * Dloc);
  float* dp = dense + batch * per + (size_t)i * Nloc + k;
  if (kExport) *dp = w_load(w, (int)batch, r, per); else w_store(w, (int)batch, r, per, *dp);
}

cudaError_t launch_weights_export(const Geom& g, const void* w, float* dense, cudaStream_t s) {
  const size_t total = (size_t)g.B * g.P * g.Nloc * g.Dloc;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (g.f32) weights_convert_kernel<float, true><<<blocks, 256, 0, s>>>((float*)w, dense, g.Nloc, g.Dloc, total);
  else weights_convert_kernel<__nv_bfloat16, true><<<blocks, 256, 0, s>>>((__nv_bfloat16*)w, dense, g.Nloc, g.Dloc, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_weights_import(const Geom& g, const float* dense, void* w, cudaStream_t s) {
  const size_t total = (size_t)g.B * g.P * g.Nloc * g.Dloc;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (g.f32) weights_convert_kernel<float, false><<<blocks, 256, 0, s>>>((float*)w, (float*)dense, g.Nloc, g.Dloc, total);
  else weights_convert_kernel<__nv_bfloat16, false><<<blocks, 256, 0, s>>>((__nv_bfloat16*)w, (float*)dense, g.Nloc, g.Dloc, total);
  count_launch();
  return cudaGetLastError();
}

}  // namespace toma
