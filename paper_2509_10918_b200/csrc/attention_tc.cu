// Attention core softmax(Q K^T / sqrt(dh)) V (Eq. 1 with tau = 1) on the sm_100a tensor
// cores, bf16 in / bf16 out, fp32 softmax and accumulation.
//
// One CTA per (batch, head, 128 queries), keys in tiles of 64; two CTAs are resident per SM.
// Warp 4 feeds K and V tiles through separate TMA rings, warp 5 issues tcgen05 MMAs, warps 0..3
// (one thread per query row) run the online softmax straight out of tensor memory:
//   S_j = Q K_j^T          -> tensor memory, two 64-column buffers; S_{j+1} is issued before the
//                             softmax of tile j has finished, so the softmax warps never wait for a
//                             round trip through the MMA warp
//   P_j = 2^(S_j*c - m)    -> written back over S_j's first 32 columns as bf16 and used as the
//                             A operand (from tensor memory) of  O += P_j V_j
//   row sums (head_dim 64) -> a second tiny MMA, P_j x ones[64 x 16], accumulates sum_k P_jk in
//                             tensor memory: exactly the bf16 P that multiplies V, so P can be
//                             produced by truncation (one byte-permute per pair, no conversion on
//                             the XU pipe) without biasing the normalised result
//   running maximum        -> O (and the row sums) are rescaled only when the maximum grew by more
//                             than 2^8; the final division by the row sum makes a stale maximum exact
//   exponentials           -> a quarter of them are a degree-3 polynomial on the FMA pipe (relative
//                             error 7.5e-5, far below bf16 resolution of P), the rest MUFU ex2
// The whole S row of a tile (64 fp32) is fetched with one tensor-memory round trip and kept in
// registers for both the maximum and the exponentials.
// Keys past the sequence end are zero-filled by TMA and masked out.
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kBM = 128;  // queries per CTA
constexpr int kBN = 64;   // keys per tile
constexpr float kRescaleThreshold = 8.0f;

template <int DH>
struct AttCfg {
  static constexpr int kStages = DH == 64 ? 4 : 2;         // K ring depth = V ring depth
  static constexpr int kChunks = DH / 64;                  // 64-column (128-byte) slabs per row
  static constexpr int kQSlab = kBM * 128;                 // 128 query rows x 128 B
  static constexpr int kKvSlab = kBN * 128;                // 64 key rows x 128 B
  static constexpr int kQBytes = kChunks * kQSlab;
  static constexpr int kKvBytes = kChunks * kKvSlab;       // one K or V tile
  static constexpr int kOnesBytes = kBN * 128;             // [64 keys][64] bf16 ones: the N chunk after V in the PV operand
  static constexpr int kSmemBytes = 1024 + kQBytes + 2 * kStages * kKvBytes + kOnesBytes + 256;
  static constexpr bool kSumMma = DH == 64;                // row sums on the tensor pipe, truncated P
  static constexpr int kTmemCols = 256;
  static constexpr int kColS = 0, kColO = 128, kColL = 128 + DH;  // S buffers at 0 and 64
};

struct Barriers {
  uint64_t q_full;
  uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
  uint64_t s_full[2], p_full[2], pv_done, o_done;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ float ex2_mufu(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for x <= ~9 on the FMA pipe: round to nearest integer with the 1.5*2^23 trick, degree-3
// near-minimax polynomial for 2^f on [-0.5, 0.5], exponent patched in with an integer add.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -126.f);
  const float t = x + 12582912.f;
  const float f = x - (t - 12582912.f);
  float p = fmaf(0.0551716648f, f, 0.2426111251f);
  p = fmaf(p, f, 0.6932609677f);
  p = fmaf(p, f, 0.9999280572f);
  return __int_as_float(__float_as_int(p) + (int)((unsigned)__float_as_int(t) << 23));
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
template <bool kMask, bool kRegSum>
__device__ __forceinline__ float chunk_exp(const uint32_t (&r)[32], uint32_t (&pk)[16], float scale, float neg_m,
                                           int first, int valid) {
  float l = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 2) {
    const float x0 = fmaf(__uint_as_float(r[e]), scale, neg_m);
    const float x1 = fmaf(__uint_as_float(r[e + 1]), scale, neg_m);
    float p0 = ex2_mufu(x0);
    float p1 = (e & 2) ? ex2_poly(x1) : ex2_mufu(x1);  // every fourth exponential on the FMA pipe
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
template <int DH, bool kMask>
__device__ __forceinline__ bool softmax_tile(uint32_t sb, uint32_t ob, float scale_log2, int valid, int j, float& m_used,
                                             float& l, uint64_t* pv_done, uint32_t pv_parity, uint32_t* dev_status, volatile int* abort_flag) {
  using C = AttCfg<DH>;
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
    if (C::kSumMma) {
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
  constexpr bool kRegSum = !C::kSumMma;
  uint32_t pk[16];
  l += chunk_exp<kMask, kRegSum>(sub32<0>(sr), pk, scale_log2, neg_m, 0, valid);
  tmem_st16(sb, pk);
  l += chunk_exp<kMask, kRegSum>(sub32<32>(sr), pk, scale_log2, neg_m, 32, valid);
  tmem_st16(sb + 16, pk);
  tmem_wait_st();
  return true;
}

template <int DH>
__global__ void __launch_bounds__(224, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, int L, int heads,
                    float scale_log2, uint32_t* dev_status) {
  using C = AttCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + C::kQBytes;
  uint8_t* sV = sK + C::kStages * C::kKvBytes;
  uint8_t* sOnes = sV + C::kStages * C::kKvBytes;
  Barriers* bar = reinterpret_cast<Barriers*>(sOnes + C::kOnesBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * kBM, h = blockIdx.y, b = blockIdx.z;
  const int nblk = (L + kBN - 1) / kBN;

  if (threadIdx.x == 0) {
    mbar_init(&bar->q_full, 1);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->k_empty[s], 1);
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->v_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->s_full[s], 1);
      mbar_init(&bar->p_full[s], 4);  // one arrival per softmax warp
    }
    mbar_init(&bar->pv_done, 1);
    mbar_init(&bar->o_done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
  }
  if (C::kSumMma) {  // bf16 1.0 everywhere: the layout's swizzle is irrelevant for a constant tile
    for (int e = threadIdx.x; e < C::kOnesBytes / 4; e += blockDim.x) reinterpret_cast<uint32_t*>(sOnes)[e] = 0x3F803F80u;
    fence_proxy_async();
  }
  if (warp == 5) tmem_alloc(&bar->tmem_base, C::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tmap(&tm_q);
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
      mbar_expect_tx(&bar->q_full, C::kQBytes);
      for (int c = 0; c < C::kChunks; ++c) tma_load_3d(sQ + c * C::kQSlab, &tm_q, &bar->q_full, h * DH + c * 64, q0, b);
      for (int j = 0; j < nblk; ++j) {
        const int s = j % C::kStages;
        const uint32_t par = ((j / C::kStages) - 1) & 1;
        if (j >= C::kStages && !mbar_wait(&bar->v_empty[s], par, dev_status, abort_flag)) break;
        mbar_expect_tx(&bar->k_full[s], 2 * C::kKvBytes);  // K and V of tile j arrive under one barrier
        for (int c = 0; c < C::kChunks; ++c)
          tma_load_3d(sK + s * C::kKvBytes + c * C::kKvSlab, &tm_k, &bar->k_full[s], h * DH + c * 64, j * kBN, b);
        for (int c = 0; c < C::kChunks; ++c)
          tma_load_3d(sV + s * C::kKvBytes + c * C::kKvSlab, &tm_v, &bar->k_full[s], h * DH + c * 64, j * kBN, b);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer for S = Q K^T
    // The two issuers are separate warps so that their waits and commits (each a serial, ~100-cycle
    // operation for a single thread) proceed in parallel.
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_f16(kFmtBF16, kFmtBF16, false, false, kBM, kBN);
      // Descriptors are built once and advanced by adding a constant to the 14-bit start-address
      // field (no carry: all tiles live below 256 KB).
      const uint64_t q_desc = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(sK), 16, 1024);
      bool ok = mbar_wait(&bar->q_full, 0, dev_status, abort_flag);
      for (int j = 0; ok && j < nblk; ++j) {
        const int s = j % C::kStages;
        if (!mbar_wait(&bar->k_full[s], (j / C::kStages) & 1, dev_status, abort_flag)) break;
        // S_j overwrites the buffer whose P_{j-2} the PV (and row-sum) MMAs of tile j-2 read as their
        // A operand.  MMAs into different accumulators are not ordered among themselves, so that read
        // has to be complete before the overwrite is issued.
        if (j >= 2 && !mbar_wait(&bar->v_empty[(j - 2) % C::kStages], ((j - 2) / C::kStages) & 1, dev_status, abort_flag)) break;
        tc_fence_after();
        const uint64_t kb = k_desc0 + (uint64_t)((s * C::kKvBytes) >> 4);
        const uint32_t t_s = tmem + C::kColS + (j & 1) * kBN;
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint64_t qoff = (uint64_t)(((kk >> 2) * C::kQSlab + (kk & 3) * 32) >> 4);
          const uint64_t koff = (uint64_t)(((kk >> 2) * C::kKvSlab + (kk & 3) * 32) >> 4);
          mma_ss(t_s, q_desc + qoff, kb + koff, idesc_s, kk > 0);
        }
        mma_commit(&bar->s_full[j & 1]);
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ MMA issuer for O += P V
    if (lane == 0) {
      // With row sums on the tensor pipe the B operand is [V | ones]: N = DH + 16, the 16 extra
      // columns come from a constant slab of ones placed one "leading byte offset" after V's slab,
      // so one MMA per 16 keys updates O and the row sums (which sit right behind O in tensor memory).
      constexpr uint32_t idesc_o = idesc_f16(kFmtBF16, kFmtBF16, false, true, kBM, C::kSumMma ? DH + 16 : DH);
      uint64_t v_desc[4];
#pragma unroll
      for (int st = 0; st < 4; ++st) {
        const int ss = st < C::kStages ? st : 0;
        const uint32_t va = smem_u32(sV + ss * C::kKvBytes);
        v_desc[st] = smem_desc_sw128(va, C::kSumMma ? smem_u32(sOnes) - va : (uint32_t)C::kKvSlab, 1024);
      }
      const uint32_t t_o = tmem + C::kColO;
      for (int j = 0; j < nblk; ++j) {
        const int s = j % C::kStages;
        if (!mbar_wait(&bar->p_full[j & 1], (j >> 1) & 1, dev_status, abort_flag)) break;  // implies K/V tile j has landed
        tc_fence_after();
        const uint64_t vb = s == 0 ? v_desc[0] : s == 1 ? v_desc[1] : s == 2 ? v_desc[2] : v_desc[3];
        const uint32_t t_p = tmem + C::kColS + (j & 1) * kBN;
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk) {  // 16 keys per MMA: 8 packed columns of P, 16 rows of V
          mma_ts(t_o, t_p + kk * 8, vb + (uint64_t)((kk * 2048) >> 4), idesc_o, j > 0 || kk > 0);
        }
        mma_commit(&bar->v_empty[s]);  // frees the K/V slot and tells everyone that PV_j has landed
        if (j + 1 == nblk) mma_commit(&bar->o_done);  // single-phase barrier: the epilogue cannot mistake an older phase for it
      }
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------------ softmax / correction / epilogue
    const int row = warp * 32 + lane;  // query row inside the tile = tensor-memory lane
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    const uint32_t ob = tmem + lane_addr + C::kColO;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nblk; ++j) {
      const uint32_t sb = tmem + lane_addr + C::kColS + (j & 1) * kBN;
      if (!mbar_wait(&bar->s_full[j & 1], (j >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int valid = L - j * kBN;  // keys of this tile inside the sequence (>= 64: all)
      uint64_t* pvb = &bar->v_empty[(j + C::kStages - 1) % C::kStages];  // barrier PV_{j-1} commits to
      const uint32_t pvp = (uint32_t)(((j - 1) / C::kStages) & 1);
      if (valid >= kBN) ok = softmax_tile<DH, false>(sb, ob, scale_log2, kBN, j, m_used, l, pvb, pvp, dev_status, abort_flag);
      else ok = softmax_tile<DH, true>(sb, ob, scale_log2, valid, j, m_used, l, pvb, pvp, dev_status, abort_flag);
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->p_full[j & 1]);
    }
    if (ok && mbar_wait(&bar->o_done, 0, dev_status, abort_flag)) {
      tc_fence_after();
      if (C::kSumMma) {
        uint32_t rs[16];
        tmem_ld16(ob + DH, rs);
        tmem_wait_ld();
        l = __uint_as_float(rs[0]);
      }
      const float inv = 1.f / l;
      const int qi = q0 + row;
      __nv_bfloat16* dst = o + ((size_t)b * L + (qi < L ? qi : 0)) * ((size_t)heads * DH) + (size_t)h * DH;
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(ob + c * 32, r);
        tmem_wait_ld();
        if (qi < L) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 v;
            v.x = pack_bf16_rn(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
            v.y = pack_bf16_rn(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            v.z = pack_bf16_rn(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            v.w = pack_bf16_rn(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + c * 32 + e) = v;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, C::kTmemCols);
  }
}

template <int DH>
cudaError_t launch(int B, int L, int heads, const void* q, const void* k, const void* v, void* o, uint32_t* dev_status,
                   cudaStream_t s) {
  using C = AttCfg<DH>;
  CUtensorMap tq, tk, tv;
  const uint64_t dims[3] = {(uint64_t)heads * DH, (uint64_t)L, (uint64_t)B};
  const uint64_t strides[2] = {(uint64_t)heads * DH * 2, (uint64_t)L * heads * DH * 2};
  const uint32_t box_q[3] = {64, kBM, 1};
  const uint32_t box_kv[3] = {64, kBN, 1};
  if (!encode_tmap_16bit(&tq, q, 3, dims, strides, box_q) || !encode_tmap_16bit(&tk, k, 3, dims, strides, box_kv) ||
      !encode_tmap_16bit(&tv, v, 3, dims, strides, box_kv))
    return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((L + kBM - 1) / kBM, heads, B);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  attention_tc_kernel<DH><<<grid, 224, C::kSmemBytes, s>>>(tq, tk, tv, (__nv_bfloat16*)o, L, heads, scale_log2, dev_status);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention_tc(int B, int L, int heads, int dh, const void* q, const void* k, const void* v, void* o,
                                uint32_t* dev_status, cudaStream_t s) {
  if (dh == 64) return launch<64>(B, L, heads, q, k, v, o, dev_status, s);
  if (dh == 128) return launch<128>(B, L, heads, q, k, v, o, dev_status, s);
  return cudaErrorInvalidValue;
}

}  // namespace toma
