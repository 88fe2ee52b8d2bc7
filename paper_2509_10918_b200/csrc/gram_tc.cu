// Fixed-point Gram matrix of one tile on the tensor cores (Sec. 4.1: the similarity matrix the
// greedy selection consumes).  Input is the quantised token directions y (bf16, tile-major
// [tile][N_loc][d]); every y is k * 2^-12 with an integer k of at most 8 significant bits and
// |y| < 1, so every partial sum of y_i . y_j is a multiple of 2^-24 below 1 and the fp32
// accumulation in tensor memory is exact whatever the order.  Output S_q[i][j] =
// rint(<y_i, y_j> * 4096) as int16, diagonal forced to 4014.
// grid (tile, 128-row block, column block of <= 256); warp 0 TMA, warp 1 MMA, warps 2..5 epilogue.
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kKC = 64;  // channels per stage
constexpr int kStages = 4;

struct GramBars {
  uint64_t full[kStages], empty[kStages], done;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(192, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               int16_t* __restrict__ sq, int Nloc, int d, int n_cols, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = 128 * 128, b_bytes = n_cols * 128;
  const int stage_bytes = a_bytes + b_bytes;
  GramBars* bar = reinterpret_cast<GramBars*>(smem + kStages * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, m0 = blockIdx.y * 128, n0 = blockIdx.z * n_cols;
  const int nk = (d + kKC - 1) / kKC;
  const uint32_t ncols = n_cols > 128 ? 256u : n_cols > 64 ? 128u : n_cols > 32 ? 64u : 32u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
  }
  dependency_wait();  // before tensor memory is held and before any global access
  if (threadIdx.x == 0) release_dependents();
  if (warp == 1) tmem_alloc(&bar->tmem_base, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 0) {
    if (elect_one()) {
      for (int k = 0; k < nk; ++k) {
        const int s = k % kStages;
        if (k >= kStages && !mbar_wait(&bar->empty[s], ((k / kStages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sa = smem + s * stage_bytes;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        tma_load_3d(sa, &tm_a, &bar->full[s], k * kKC, m0, tile);
        tma_load_3d(sa + a_bytes, &tm_b, &bar->full[s], k * kKC, n0, tile);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, n_cols);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % kStages;
        if (!mbar_wait(&bar->full[s], (k / kStages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t aa = smem_u32(smem + s * stage_bytes), ba = aa + a_bytes;
#pragma unroll
        for (int kk = 0; kk < kKC / 16; ++kk)
          mma_ss(tmem, smem_desc_sw128(aa + kk * 32, 16, 1024), smem_desc_sw128(ba + kk * 32, 16, 1024), idesc,
                 k > 0 || kk > 0);
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3;
    const int i = m0 + quarter * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    if (mbar_wait(&bar->done, 0, dev_status, abort_flag)) {
      tc_fence_after();
      int16_t* row = sq + ((size_t)tile * Nloc + (i < Nloc ? i : 0)) * Nloc + n0;
      for (int j0 = 0; j0 < n_cols; j0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + j0, r);
        tmem_wait_ld();
        if (i < Nloc) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            if (j0 + e >= n_cols) break;
            uint32_t pk[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int ja = n0 + j0 + e + 2 * u;
              int lo = __float2int_rn(__uint_as_float(r[e + 2 * u]) * 4096.f);
              int hi = __float2int_rn(__uint_as_float(r[e + 2 * u + 1]) * 4096.f);
              if (ja == i) lo = kDiagQ;
              if (ja + 1 == i) hi = kDiagQ;
              pk[u] = ((uint32_t)hi << 16) | ((uint32_t)lo & 0xFFFFu);
            }
            *reinterpret_cast<uint4*>(row + j0 + e) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

}  // namespace

bool gram_tc_supported(const Geom& g) {
  if (g.Nloc % 16 != 0) return false;
  if (g.Nloc > 256 && g.Nloc % 256 != 0) return false;
  return true;
}

cudaError_t launch_gram_tc(const Geom& g, const __nv_bfloat16* y, int16_t* sq, uint32_t* dev_status, cudaStream_t s) {
  const int n_cols = g.Nloc > 256 ? 256 : g.Nloc;
  CUtensorMap ta, tb;
  const uint64_t dims[3] = {(uint64_t)g.d, (uint64_t)g.Nloc, (uint64_t)g.B * g.P};
  const uint64_t strides[2] = {(uint64_t)g.d * 2, (uint64_t)g.Nloc * g.d * 2};
  const uint32_t box_a[3] = {64, 128, 1};
  const uint32_t box_b[3] = {64, (uint32_t)n_cols, 1};
  if (!encode_tmap_16bit(&ta, y, 3, dims, strides, box_a) || !encode_tmap_16bit(&tb, y, 3, dims, strides, box_b))
    return cudaErrorInvalidValue;
  const int smem = 1024 + kStages * (128 * 128 + n_cols * 128) + 256;
  static std::atomic<unsigned long long> smem_raised{0};
  if (cudaError_t e = raise_dynamic_smem(gram_tc_kernel, 200 * 1024, smem_raised); e != cudaSuccess) return e;
  dim3 grid(g.B * g.P, (g.Nloc + 127) / 128, g.Nloc / n_cols);
  const cudaError_t le = launch_dependent(gram_tc_kernel, grid, dim3(192), (size_t)smem, s, ta, tb, sq, g.Nloc, g.d, n_cols, dev_status);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace toma
