// Attention core softmax(Q K^T / sqrt(dh)) V (Eq. 1 with tau = 1) on the sm_100a tensor
// cores, bf16 in / bf16 out, fp32 softmax and accumulation.
//
// One CTA per (batch, head, 128 queries).  Warp 0 feeds K/V tiles of 128 keys through a TMA
// ring, warp 1 issues tcgen05 MMAs, warps 2..5 (one thread per query row) run the online
// softmax straight out of tensor memory:
//   S_j = Q K_j^T          -> tensor memory, double buffered, issued one tile ahead
//   P_j = 2^(S_j*c - m)    -> written back over S_j's columns as bf16 (A operand from tensor memory)
//   O  += P_j V_j          -> tensor memory accumulator; rescaled only when the running maximum
//                             grew by more than 2^8 (the final division by the row sum makes the
//                             stale maximum exact)
// Keys past the sequence end are zero-filled by TMA and masked to -inf.
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kBM = 128;  // queries per CTA
constexpr int kBN = 128;  // keys per tile
constexpr float kRescaleThreshold = 8.0f;

template <int DH>
struct AttCfg {
  static constexpr int kStages = DH == 64 ? 3 : 2;
  static constexpr int kChunks = DH / 64;                 // 64-column (128-byte) slabs per row
  static constexpr int kSlabBytes = 128 * 128;            // 128 rows x 128 B
  static constexpr int kTileBytes = kChunks * kSlabBytes; // one Q, K or V tile
  static constexpr int kSmemBytes = 1024 + kTileBytes * (1 + 2 * kStages) + 256;
  static constexpr int kTmemCols = 512;
  static constexpr int kColS0 = 0, kColS1 = 128, kColO = 256;
};

struct Barriers {
  uint64_t q_full;
  uint64_t k_full[3], v_full[3], kv_empty[3];
  uint64_t s_full[2], p_full[2];
  uint64_t o_done;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int DH>
__global__ void __launch_bounds__(192, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, int L, int heads,
                    float scale_log2, uint32_t* dev_status) {
  using C = AttCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + C::kTileBytes;
  uint8_t* sV = sK + C::kStages * C::kTileBytes;
  Barriers* bar = reinterpret_cast<Barriers*>(sV + C::kStages * C::kTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * kBM, h = blockIdx.y, b = blockIdx.z;
  const int nblk = (L + kBN - 1) / kBN;

  if (threadIdx.x == 0) {
    mbar_init(&bar->q_full, 1);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->kv_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->s_full[s], 1);
      mbar_init(&bar->p_full[s], 128);
    }
    mbar_init(&bar->o_done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&bar->tmem_base, C::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tmap(&tm_q);
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
      mbar_expect_tx(&bar->q_full, C::kTileBytes);
      for (int c = 0; c < C::kChunks; ++c) tma_load_3d(sQ + c * C::kSlabBytes, &tm_q, &bar->q_full, h * DH + c * 64, q0, b);
      for (int j = 0; j < nblk; ++j) {
        const int s = j % C::kStages;
        if (j >= C::kStages && !mbar_wait(&bar->kv_empty[s], ((j / C::kStages) - 1) & 1, dev_status, abort_flag)) break;
        mbar_expect_tx(&bar->k_full[s], C::kTileBytes);
        for (int c = 0; c < C::kChunks; ++c)
          tma_load_3d(sK + s * C::kTileBytes + c * C::kSlabBytes, &tm_k, &bar->k_full[s], h * DH + c * 64, j * kBN, b);
        mbar_expect_tx(&bar->v_full[s], C::kTileBytes);
        for (int c = 0; c < C::kChunks; ++c)
          tma_load_3d(sV + s * C::kTileBytes + c * C::kSlabBytes, &tm_v, &bar->v_full[s], h * DH + c * 64, j * kBN, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_f16(kFmtBF16, kFmtBF16, false, false, kBM, kBN);
      constexpr uint32_t idesc_o = idesc_f16(kFmtBF16, kFmtBF16, false, true, kBM, DH);
      auto issue_s = [&](int j) {  // S_j = Q K_j^T
        const int s = j % C::kStages;
        const uint32_t d = tmem + ((j & 1) ? C::kColS1 : C::kColS0);
        const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK + s * C::kTileBytes);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t off = (kk >> 2) * C::kSlabBytes + (kk & 3) * 32;
          mma_ss(d, smem_desc_sw128(qa + off, 16, 1024), smem_desc_sw128(ka + off, 16, 1024), idesc_s, kk > 0);
        }
        mma_commit(&bar->s_full[j & 1]);
      };
      bool ok = mbar_wait(&bar->q_full, 0, dev_status, abort_flag) && mbar_wait(&bar->k_full[0], 0, dev_status, abort_flag);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; ok && j < nblk; ++j) {
        const int s = j % C::kStages;
        if (j + 1 < nblk) {
          const int s1 = (j + 1) % C::kStages;
          if (!mbar_wait(&bar->k_full[s1], ((j + 1) / C::kStages) & 1, dev_status, abort_flag)) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        if (!mbar_wait(&bar->p_full[j & 1], (j >> 1) & 1, dev_status, abort_flag)) break;
        if (!mbar_wait(&bar->v_full[s], (j / C::kStages) & 1, dev_status, abort_flag)) break;
        tc_fence_after();
        const uint32_t pa = tmem + ((j & 1) ? C::kColS1 : C::kColS0);
        const uint32_t va = smem_u32(sV + s * C::kTileBytes);
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk)  // 16 keys per MMA: 8 packed columns of P, 16 rows of V
          mma_ts(tmem + C::kColO, pa + kk * 8, smem_desc_sw128(va + kk * 2048, C::kSlabBytes, 1024), idesc_o,
                 j > 0 || kk > 0);
        mma_commit(&bar->kv_empty[s]);
        mma_commit(&bar->o_done);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / correction / epilogue
    const int quarter = warp & 3;              // tensor-memory lane quarter this warp may access
    const int row = quarter * 32 + lane;       // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nblk; ++j) {
      const uint32_t sb = tmem + lane_addr + ((j & 1) ? C::kColS1 : C::kColS0);
      if (!mbar_wait(&bar->s_full[j & 1], (j >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int valid = min(kBN, L - j * kBN);  // keys of this tile inside the sequence
      // pass 1: row maximum
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(sb + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float v = __uint_as_float(r[e]);
          mx = fmaxf(mx, (c * 32 + e < valid) ? v : -INFINITY);
        }
      }
      mx *= scale_log2;
      float factor = 1.f;
      bool rescale = false;
      if (j == 0) {
        m_used = mx;
      } else if (mx > m_used + kRescaleThreshold) {
        factor = fast_exp2(m_used - mx);
        m_used = mx;
        rescale = true;
      }
      if (__any_sync(0xffffffffu, rescale)) {
        // O holds every PV product issued so far; wait for the last one before touching it
        if (!mbar_wait(&bar->o_done, (j - 1) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        l *= factor;
#pragma unroll
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + C::kColO + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * factor);
          tmem_st32(tmem + lane_addr + C::kColO + c * 32, r);
        }
      }
      // pass 2: P = 2^(S*c - m), packed bf16 written over the first 64 columns of S_j
      const float neg_m = -m_used;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(sb + c * 32, r);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float p0 = fast_exp2(fmaf(__uint_as_float(r[e]), scale_log2, neg_m));
          float p1 = fast_exp2(fmaf(__uint_as_float(r[e + 1]), scale_log2, neg_m));
          if (c * 32 + e >= valid) p0 = 0.f;
          if (c * 32 + e + 1 >= valid) p1 = 0.f;
          l += p0 + p1;
          pk[e >> 1] = pack_bf16(p0, p1);
        }
        tmem_st16(sb + c * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar->p_full[j & 1]);
    }
    if (ok && mbar_wait(&bar->o_done, (nblk - 1) & 1, dev_status, abort_flag)) {
      tc_fence_after();
      const float inv = 1.f / l;
      const int qi = q0 + row;
      __nv_bfloat16* dst = o + ((size_t)b * L + (qi < L ? qi : 0)) * ((size_t)heads * DH) + (size_t)h * DH;
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_addr + C::kColO + c * 32, r);
        tmem_wait_ld();
        if (qi < L) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + c * 32 + e) = v;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
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
  const uint32_t box[3] = {64, 128, 1};
  if (!encode_tmap_16bit(&tq, q, 3, dims, strides, box) || !encode_tmap_16bit(&tk, k, 3, dims, strides, box) ||
      !encode_tmap_16bit(&tv, v, 3, dims, strides, box))
    return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((L + kBM - 1) / kBM, heads, B);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  attention_tc_kernel<DH><<<grid, 192, C::kSmemBytes, s>>>(tq, tk, tv, (__nv_bfloat16*)o, L, heads, scale_log2, dev_status);
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
