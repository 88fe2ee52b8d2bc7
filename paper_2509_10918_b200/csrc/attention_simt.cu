// FFMA attention core softmax(Q K^T / sqrt(dh)) V (Eq. 1 with tau = 1) with an
// online softmax.  64 queries per CTA, four threads per query, each owning a
// quarter of the head dimension; keys/values are staged 32 at a time in shared
// memory as fp32.  Used for the fp32 mode and for head sizes the tensor-core
// kernel does not cover.
#include "common.cuh"

namespace toma {

template <typename T, int DH>
__global__ void __launch_bounds__(256) attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                             const T* __restrict__ v, T* __restrict__ o, int L,
                                                             int heads, float scale) {
  constexpr int SEG = DH / 4;  // channels per thread
  constexpr int KT = 32;       // keys per tile
  __shared__ __align__(16) float Ks[KT][DH];
  __shared__ __align__(16) float Vs[KT][DH];
  const int b = blockIdx.z, h = blockIdx.y;
  const int ql = threadIdx.x >> 2, part = threadIdx.x & 3;
  const int qi = blockIdx.x * 64 + ql;
  const size_t row_stride = (size_t)heads * DH;
  const size_t base = (size_t)b * L * row_stride + (size_t)h * DH;
  float qr[SEG], acc[SEG];
  const int qsafe = qi < L ? qi : L - 1;
#pragma unroll
  for (int c = 0; c < SEG; ++c) {
    qr[c] = to_f32(q[base + (size_t)qsafe * row_stride + part * SEG + c]) * scale;
    acc[c] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  for (int k0 = 0; k0 < L; k0 += KT) {
    __syncthreads();
    for (int e = threadIdx.x; e < KT * DH; e += 256) {
      const int r = e / DH, c = e - r * DH;
      const bool in = k0 + r < L;
      Ks[r][c] = in ? to_f32(k[base + (size_t)(k0 + r) * row_stride + c]) : 0.f;
      Vs[r][c] = in ? to_f32(v[base + (size_t)(k0 + r) * row_stride + c]) : 0.f;
    }
    __syncthreads();
    float s[KT];
    float tmax = -INFINITY;
#pragma unroll
    for (int r = 0; r < KT; ++r) {
      float part_dot = 0.f;
#pragma unroll
      for (int c = 0; c < SEG; c += 4) {
        const float4 kk = *reinterpret_cast<const float4*>(&Ks[r][part * SEG + c]);
        part_dot = fmaf(qr[c], kk.x, part_dot);
        part_dot = fmaf(qr[c + 1], kk.y, part_dot);
        part_dot = fmaf(qr[c + 2], kk.z, part_dot);
        part_dot = fmaf(qr[c + 3], kk.w, part_dot);
      }
      part_dot += __shfl_xor_sync(0xffffffffu, part_dot, 1);
      part_dot += __shfl_xor_sync(0xffffffffu, part_dot, 2);
      s[r] = (k0 + r < L) ? part_dot : -INFINITY;
      tmax = fmaxf(tmax, s[r]);
    }
    const float m_new = fmaxf(m, tmax);
    const float corr = expf(m - m_new);  // m = -inf on the first tile gives 0
    l *= corr;
#pragma unroll
    for (int c = 0; c < SEG; ++c) acc[c] *= corr;
#pragma unroll
    for (int r = 0; r < KT; ++r) {
      const float p = expf(s[r] - m_new);
      l += p;
#pragma unroll
      for (int c = 0; c < SEG; c += 4) {
        const float4 vv = *reinterpret_cast<const float4*>(&Vs[r][part * SEG + c]);
        acc[c] = fmaf(p, vv.x, acc[c]);
        acc[c + 1] = fmaf(p, vv.y, acc[c + 1]);
        acc[c + 2] = fmaf(p, vv.z, acc[c + 2]);
        acc[c + 3] = fmaf(p, vv.w, acc[c + 3]);
      }
    }
    m = m_new;
  }
  if (qi < L) {
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < SEG; ++c) from_f32(o[base + (size_t)qi * row_stride + part * SEG + c], acc[c] * inv);
  }
}

template <typename T>
static cudaError_t run(int B, int L, int heads, int dh, const void* q, const void* k, const void* v, void* o,
                       cudaStream_t s) {
  dim3 grid((L + 63) / 64, heads, B);
  const float scale = 1.0f / sqrtf((float)dh);
#define TOMA_ATT_CASE(D)                                                                                        \
  case D:                                                                                                       \
    attention_simt_kernel<T, D><<<grid, 256, 0, s>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, L, heads, scale); \
    break;
  switch (dh) {
    TOMA_ATT_CASE(16)
    TOMA_ATT_CASE(32)
    TOMA_ATT_CASE(64)
    TOMA_ATT_CASE(128)
    default:
      return cudaErrorInvalidValue;
  }
#undef TOMA_ATT_CASE
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_attention_simt(int B, int L, int heads, int dh, bool f32, const void* q, const void* k,
                                  const void* v, void* o, cudaStream_t s) {
  return f32 ? run<float>(B, L, heads, dh, q, k, v, o, s) : run<__nv_bfloat16>(B, L, heads, dh, q, k, v, o, s);
}

}  // namespace toma
