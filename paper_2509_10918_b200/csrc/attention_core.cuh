// Device helpers of the tensor-core attention kernels: the online softmax of one 64-key tile for one
// query row straight out of tensor memory (see attention_tc.cu for the scheme), and the scaled bf16
// store of accumulator rows.
#pragma once

#include "common.cuh"
#include "tc.cuh"

namespace toma {
namespace attn {

using namespace tc;

constexpr int kBM = 128;  // rows of one query tile = threads of one softmax warp group
constexpr int kBN = 64;   // keys per tile
constexpr float kRescaleThreshold = 8.0f;

__device__ __forceinline__ float ex2_mufu(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Two floats in one 64-bit register and the packed fp32 arithmetic of sm_100 on them (one issue slot for two
// results on the FMA pipe).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for x <= ~9 on the FMA pipe, two at a time: round to nearest integer with the 1.5*2^23 trick, degree-3
// near-minimax polynomial for 2^f on [-0.5, 0.5], exponent patched in with an integer add.
__device__ __forceinline__ void ex2_poly2(uint64_t x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  x2 = pack2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const uint64_t k2 = pack2(12582912.f, 12582912.f);
  const uint64_t t2 = add2(x2, k2);
  const uint64_t f2 = sub2(x2, sub2(t2, k2));
  uint64_t q2 = fma2(pack2(0.0551716648f, 0.0551716648f), f2, pack2(0.2426111251f, 0.2426111251f));
  q2 = fma2(q2, f2, pack2(0.6932609677f, 0.6932609677f));
  q2 = fma2(q2, f2, pack2(0.9999280572f, 0.9999280572f));
  float q0, q1, t0, t1;
  unpack2(q2, q0, q1);
  unpack2(t2, t0, t1);
  p0 = __int_as_float(__float_as_int(q0) + (int)((unsigned)__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (int)((unsigned)__float_as_int(t1) << 23));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16_rn(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16_trunc(float lo, float hi) {  // upper halves of both words
  return __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x7632);
}

// View of 32 consecutive registers of a larger per-thread array (all indices are compile-time).
template <int kOff, int kN>
__device__ __forceinline__ uint32_t (&sub32(uint32_t (&r)[kN]))[32] {
  return *reinterpret_cast<uint32_t(*)[32]>(&r[kOff]);
}

// Maximum of 32 tensor-memory words (columns first .. first+31 of this row; columns >= valid ignored).
template <bool kMask>
__device__ __forceinline__ float chunk_max(const uint32_t (&r)[32], float mx, int first, int valid) {
  if (kMask) {
#pragma unroll
    for (int e = 0; e < 32; ++e) mx = fmaxf(mx, (first + e < valid) ? __uint_as_float(r[e]) : -INFINITY);
  } else {
#pragma unroll
    for (int e = 0; e < 32; e += 2) mx = max3(mx, __uint_as_float(r[e]), __uint_as_float(r[e + 1]));
  }
  return mx;
}

// P for 32 columns as packed bf16 pairs in pk[16]; returns their fp32 sum when sums stay in registers.
// kMorePoly: three pairs of columns in eight instead of two take the polynomial (timed: 1-2 % faster at head_dim
// 128, where the sums add to the FMA pipe's load anyway, 4 % slower at head_dim 64).
template <bool kMask, bool kRegSum, bool kMorePoly>
__device__ __forceinline__ float chunk_exp(const uint32_t (&r)[32], uint32_t (&pk)[16], float scale, float neg_m,
                                           int first, int valid) {
  float l = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 2) {
    // S * c - m for a pair of columns in one packed multiply-add
    const uint64_t x2 = fma2(pack2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), pack2(scale, scale), pack2(neg_m, neg_m));
    float p0, p1;
    const bool poly = kMorePoly ? ((e & 14) == 6 || (e & 14) == 10 || (e & 14) == 14) : (e & 6) == 6;
    if (poly) {  // this pair of exponentials on the FMA pipe
      ex2_poly2(x2, p0, p1);
    } else {
      float x0, x1;
      unpack2(x2, x0, x1);
      p0 = ex2_mufu(x0);
      p1 = ex2_mufu(x1);
    }
    if (kMask) {
      if (first + e >= valid) p0 = 0.f;
      if (first + e + 1 >= valid) p1 = 0.f;
    }
    if (kRegSum) {
      l += p0 + p1;
      pk[e >> 1] = pack_bf16_rn(p0, p1);
    } else {
      pk[e >> 1] = pack_bf16_trunc(p0, p1);
    }
  }
  return l;
}

// One 64-key tile of the online softmax for one query row.
template <int DH, bool kSumMma, bool kMask>
__device__ __forceinline__ bool softmax_tile(uint32_t sb, uint32_t ob, float scale_log2, int valid, int j, float& m_used,
                                             float& l, uint64_t* pv_done, uint32_t pv_parity, uint32_t* dev_status, volatile int* abort_flag) {
  uint32_t sr[64];
  tmem_ld32(sb, sub32<0>(sr));
  tmem_ld32(sb + 32, sub32<32>(sr));
  tmem_wait_ld();
  float mx = -INFINITY;
  mx = chunk_max<kMask>(sub32<0>(sr), mx, 0, valid);
  mx = chunk_max<kMask>(sub32<32>(sr), mx, 32, valid);
  mx *= scale_log2;
  float factor = 1.f;
  bool rescale = false;
  if (j == 0) {
    m_used = mx;
  } else if (mx > m_used + kRescaleThreshold) {
    factor = ex2_mufu(m_used - mx);
    m_used = mx;
    rescale = true;
  }
  if (__any_sync(0xffffffffu, rescale)) {
    // O holds every PV product issued so far; the last one (tile j-1) must have landed
    if (!mbar_wait(pv_done, pv_parity, dev_status, abort_flag)) return false;
    tc_fence_after();
    l *= factor;
#pragma unroll
    for (int c = 0; c < DH / 32; ++c) {
      uint32_t t[32];
      tmem_ld32(ob + c * 32, t);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) t[e] = __float_as_uint(__uint_as_float(t[e]) * factor);
      tmem_st32(ob + c * 32, t);
    }
    if (kSumMma) {
      uint32_t rs[16];
      tmem_ld16(ob + DH, rs);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) rs[e] = __float_as_uint(__uint_as_float(rs[e]) * factor);
      tmem_st16(ob + DH, rs);
    }
  }
  // P = 2^(S*c - m) as packed bf16 over the first 32 columns of this S buffer
  const float neg_m = -m_used;
  constexpr bool kRegSum = !kSumMma;
  uint32_t pk[16];
  l += chunk_exp<kMask, kRegSum, DH == 128>(sub32<0>(sr), pk, scale_log2, neg_m, 0, valid);
  tmem_st16(sb, pk);
  l += chunk_exp<kMask, kRegSum, DH == 128>(sub32<32>(sr), pk, scale_log2, neg_m, 32, valid);
  tmem_st16(sb + 16, pk);
  tmem_wait_st();
  return true;
}

// 32 accumulator columns of one row, scaled and rounded to bf16: 64 contiguous bytes.
__device__ __forceinline__ void store_row32(__nv_bfloat16* dst, const uint32_t (&r)[32], float inv) {
#pragma unroll
  for (int e = 0; e < 32; e += 8) {
    uint4 v;
    v.x = pack_bf16_rn(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
    v.y = pack_bf16_rn(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
    v.z = pack_bf16_rn(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
    v.w = pack_bf16_rn(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
    *reinterpret_cast<uint4*>(dst + e) = v;
  }
}

}  // namespace attn
}  // namespace toma
