// Dense projection C[m][n] = sum_k A[m][k] W[k][n] on the sm_100a tensor cores (bf16 in, fp32
// accumulation in tensor memory, bf16 out): the QKV and output projections of the attention module
// that ToMA wraps (Algorithm 3's core module F; App. C counts them as the 4 d^2 N term).
//
// Rows of A (tokens) sit on the MMA M dimension, 128 per CTA; a CTA covers up to 320 output columns
// (two MMAs along N, at most 192 + 128).  A is the K-major operand exactly as stored ([m][k] row-major),
// W the MN-major one exactly as stored ([k][n] row-major), so neither is transposed or copied.
// blockIdx.z selects one of up to three weight / output pairs that share A (Q, K and V in one
// launch).  Warp 0 feeds a TMA ring, warp 1 issues the MMAs, warps 2..5 take the accumulators out of tensor
// memory (through the activation when one is asked for: the first layer of the MLP, the other module ToMA
// wraps), stage each warp's 32 rows in shared memory as 64-column slabs in the layout of the output tensor
// map's box (the ring is free by then) and store them with one TMA store per warp and slab: whole lines,
// asynchronous, instead of 16-byte stores to 32 different rows per warp instruction.
#include <cstdlib>

#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kKC = 64;                  // contraction elements per stage
constexpr int kSlab = kKC * 128;         // [64 k][64 n] slab of W, 128-byte rows
constexpr int kABytes = 128 * 128;       // [128 m][64 k] slab of A

struct GemmBars {
  uint64_t full[4], empty[4], done;
  uint32_t tmem_base;
  int abort_flag;
};


// kCols = 320: two accumulators (192 + 128 columns), 512 tensor-memory columns, one CTA per SM, deep ring.
// kCols = 256: one accumulator, 256 tensor-memory columns, two CTAs per SM, for grids that would otherwise
// spill into a second wave or leave most SMs idle.
// kCols = 128: 128 tensor-memory columns and 32 KB stages, two CTAs per SM, for narrow outputs with a long
// contraction (the second layer of the MLP: 4096 x 640 x 2560 is 64 tiles of 128 x 320 but 160 of 128 x 128).
// kRowBlocks = 2 (with kCols = 256): two 128-row blocks per CTA share every W slab, so a CTA moves 64 KB
// per 256 x 256 x 64 multiply-adds instead of 48 KB per 128 x 256 x 64 (these shapes re-read their operands
// from L2 many times and are bound by that traffic); one CTA per SM.
template <int kCols, int kRowBlocks = 1>
__global__ void __launch_bounds__(192, 1)
linear_rows_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w0,
                   const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2,
                   const __grid_constant__ CUtensorMap tm_c0, const __grid_constant__ CUtensorMap tm_c1,
                   const __grid_constant__ CUtensorMap tm_c2, int M, int N, int K, int stages, int ring_bytes, int act,
                   uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kFirst = kCols == 320 ? 3 : 4;  // 64-column slabs of the first accumulator
  const int m0 = blockIdx.x * 128 * kRowBlocks, n0 = blockIdx.y * kCols;
  const CUtensorMap* tm_w = blockIdx.z == 0 ? &tm_w0 : blockIdx.z == 1 ? &tm_w1 : &tm_w2;
  const CUtensorMap* tm_c = blockIdx.z == 0 ? &tm_c0 : blockIdx.z == 1 ? &tm_c1 : &tm_c2;
  const int n_cols = min(kCols, N - n0);         // columns of this CTA (multiple of 8)
  const int slabs = (n_cols + 63) / 64;
  const int n_a = min(slabs, kFirst) * 64, n_b = (slabs - min(slabs, kFirst)) * 64;
  const int stage_bytes = kRowBlocks * kABytes + slabs * kSlab;
  GemmBars* bar = reinterpret_cast<GemmBars*>(smem + ring_bytes);  // behind the ring and the output's staging area, whichever is larger
  const int nk = (K + kKC - 1) / kKC;
  constexpr uint32_t ncols = (kCols == 320 || kRowBlocks == 2) ? 512 : kCols == 128 ? 128 : 256;
  static_assert(kRowBlocks == 1 || kCols == 256, "two row blocks need the one-accumulator column form");

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(tm_w);
    prefetch_tmap(tm_c);
  }
  dependency_wait();
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
        const int s = k % stages;
        if (k >= stages && !mbar_wait(&bar->empty[s], ((k / stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sa = smem + s * stage_bytes;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        for (int rb = 0; rb < kRowBlocks; ++rb) tma_load_2d(sa + rb * kABytes, &tm_a, &bar->full[s], k * kKC, m0 + rb * 128);
        for (int j = 0; j < slabs; ++j)
          tma_load_2d(sa + kRowBlocks * kABytes + j * kSlab, tm_w, &bar->full[s], n0 + j * 64, k * kKC);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc_a = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_a);
      const uint32_t idesc_b = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_b > 0 ? n_b : 64);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % stages;
        if (!mbar_wait(&bar->full[s], (k / stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t aa = smem_u32(smem + s * stage_bytes), wa = aa + kRowBlocks * kABytes;
        const int ksteps = min(kKC, K - k * kKC + 15) / 16;  // 16 contraction elements per MMA (zero filled past K)
        for (int kk = 0; kk < ksteps; ++kk) {
          const uint64_t wd = smem_desc_sw128(wa + kk * 2048, kSlab, 1024);
#pragma unroll
          for (int rb = 0; rb < kRowBlocks; ++rb) {
            const uint64_t ad = smem_desc_sw128(aa + rb * kABytes + kk * 32, 16, 1024);
            mma_ss(tmem + rb * 256, ad, wd, idesc_a, k > 0 || kk > 0);
            if (kRowBlocks == 1 && n_b > 0)
              mma_ss(tmem + kFirst * 64, ad, smem_desc_sw128(wa + kFirst * kSlab + kk * 2048, kSlab, 1024), idesc_b, k > 0 || kk > 0);
          }
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3, r_in = quarter * 32 + lane;  // row inside a 128-row block = tensor-memory lane
    // one answer per warp: the tensor-memory loads below are warp-wide operations
    if (__all_sync(0xffffffffu, mbar_wait(&bar->done, 0, dev_status, abort_flag))) {
      tc_fence_after();
      // every load has been consumed: slab j of row block rb goes to smem + (rb * slabs + j) * 16 KB as
      // [128 rows][128 B], 128-byte swizzled; a warp's 32 rows are 4 KB of it
#pragma unroll 1
      for (int rb = 0; rb < kRowBlocks; ++rb) {
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + rb * 256;
        for (int j = 0; j < n_cols; j += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + j, r);
          tmem_wait_ld();
          if (act == kActGelu) {
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(gelu(__uint_as_float(r[e])));
          }
          uint8_t* slab = smem + (rb * slabs + (j >> 6)) * (128 * 128);
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            __align__(16) __nv_bfloat162 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              q[u] = __floats2bfloat162_rn(__uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1]));
            *reinterpret_cast<uint4*>(slab + sw128_offset(r_in, ((j & 63) + e) >> 3)) = *reinterpret_cast<const uint4*>(q);
          }
        }
      }
      fence_proxy_async();  // the staged rows are read by the TMA engine
      __syncwarp();
      if (lane == 0) {
        for (int rb = 0; rb < kRowBlocks; ++rb) {
          const int row0 = m0 + rb * 128 + quarter * 32;
          if (row0 >= M) continue;  // rows past M and columns past N inside a box are clipped by the store
          for (int j = 0; j < slabs; ++j)
            tma_store_2d(tm_c, smem + (rb * slabs + j) * (128 * 128) + quarter * 4096, n0 + j * 64, row0);
        }
        tma_store_commit();
        tma_store_wait_read();  // shared memory must outlive the engine's reads
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

bool linear_tc_shape_ok(int M, int N, int K) { return M >= 1 && N >= 8 && K >= 8 && N % 8 == 0 && K % 8 == 0; }

// c[i] = a * w[i] for i < n_mats (1..3); a [M][K], w[i] [K][N], c[i] [M][N], all bf16 row-major.
cudaError_t launch_linear_tc(int M, int N, int K, const void* a, const void* const* w, void* const* c, int n_mats, int act,
                             uint32_t* dev_status, cudaStream_t s) {
  CUtensorMap ta, tw[3], tc_[3];
  const uint64_t adims[2] = {(uint64_t)K, (uint64_t)M};
  const uint64_t astr[1] = {(uint64_t)K * 2};
  const uint32_t abox[2] = {64, 128};
  if (!encode_tmap_16bit(&ta, a, 2, adims, astr, abox)) return cudaErrorInvalidValue;
  const uint64_t wdims[2] = {(uint64_t)N, (uint64_t)K};
  const uint64_t wstr[1] = {(uint64_t)N * 2};
  const uint32_t wbox[2] = {64, 64};
  const uint64_t cdims[2] = {(uint64_t)N, (uint64_t)M};
  const uint32_t cbox[2] = {64, 32};  // a warp's 32 rows of one 64-column slab
  for (int i = 0; i < 3; ++i) {
    const int j = i < n_mats ? i : 0;
    if (!encode_tmap_16bit(&tw[i], w[j], 2, wdims, wstr, wbox) || !encode_tmap_16bit(&tc_[i], c[j], 2, cdims, wstr, cbox))
      return cudaErrorInvalidValue;
  }
  // Tile form: the one with the least serial work per SM, counted as CTAs per SM (rounded up) times the
  // multiply-adds of a tile, the 256 x 256 form credited with the 1.3x it gains from moving fewer operand
  // bytes per multiply-add (timed on eleven shapes from 4096 x 640 x 640 to 16384 x 8192 x 4096; the
  // model picks the faster form on each).  The 128 x 256 form keeps two CTAs per SM resident and is only
  // considered while its grid fits them.
  const int sms = sm_count();
  const int mb = (M + 127) / 128;
  const long long ctas320 = (long long)mb * ((N + 319) / 320) * n_mats, ctas256 = (long long)mb * ((N + 255) / 256) * n_mats;
  const long long ctas_pair = (long long)((M + 255) / 256) * ((N + 255) / 256) * n_mats;
  const long long cost320 = ((ctas320 + sms - 1) / sms) * (128 * 320) * 13;
  const long long cost256 = ctas256 <= 2 * sms ? ((ctas256 + sms - 1) / sms) * (128 * 256) * 13 : cost320 + 1;
  const long long cost_pair = M > 128 ? ((ctas_pair + sms - 1) / sms) * (256 * 256) * 10 : cost320 + 1;
  // 128 x 128 tiles, two CTAs per SM sharing its tensor pipe: serial work = CTAs per SM (rounded up) tiles
  const long long ctas128 = (long long)mb * ((N + 127) / 128) * n_mats;
  const long long cost128 = ctas128 <= 2 * sms ? ((ctas128 + sms - 1) / sms) * (128 * 128) * 13 : cost320 + 1;
  // ties go to the form with more, smaller CTAs (more SMs take in operands at once)
  bool small = cost128 <= cost256 && cost128 <= cost_pair && cost128 < cost320;
  bool narrow = !small && cost256 <= cost_pair && cost256 < cost320;
  int pair = !small && !narrow && cost_pair < cost320;
  if (const int v = g_tune_linear_tile.load(std::memory_order_relaxed)) {  // test-only override: 128 x 256 (1), 128 x 320 (2), 256 x 256 (3) or 128 x 128 (4) tiles
    pair = v == 3 && M > 128;
    narrow = v == 1;
    small = v == 4;
  }
  const int cols = small ? 128 : (narrow || pair) ? 256 : 320;
  const int slabs = ((N < cols ? N : cols) + 63) / 64;
  const int stage_bytes = (pair ? 2 : 1) * kABytes + slabs * kSlab;
  int stages = (((narrow && !pair) || small ? 110 : 222) * 1024) / stage_bytes;
  stages = stages > 4 ? 4 : stages < 1 ? 1 : stages;
  const int nk = (K + kKC - 1) / kKC;
  if (stages > nk) stages = nk;
  const int staging = (pair ? 2 : 1) * slabs * 128 * 128;  // the output tile, staged where the ring was
  const int ring_bytes = stages * stage_bytes > staging ? stages * stage_bytes : staging;
  const int smem = 1024 + ring_bytes + 256;
  {
    static std::atomic<unsigned long long> r320{0}, r256{0}, rpair{0}, r128{0};
    cudaError_t e = raise_dynamic_smem(linear_rows_kernel<320>, 227 * 1024, r320);
    if (e == cudaSuccess) e = raise_dynamic_smem(linear_rows_kernel<128>, 227 * 1024, r128);
    if (e == cudaSuccess) e = raise_dynamic_smem(linear_rows_kernel<256>, 227 * 1024, r256);
    if (e == cudaSuccess) e = raise_dynamic_smem(linear_rows_kernel<256, 2>, 227 * 1024, rpair);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(pair ? (M + 255) / 256 : mb, (N + cols - 1) / cols, n_mats);
  cudaError_t e = pair ? launch_dependent(linear_rows_kernel<256, 2>, grid, dim3(192), (size_t)smem, s, ta, tw[0], tw[1], tw[2], tc_[0], tc_[1],
                                          tc_[2], M, N, K, stages, ring_bytes, act, dev_status)
                  : small ? launch_dependent(linear_rows_kernel<128>, grid, dim3(192), (size_t)smem, s, ta, tw[0], tw[1], tw[2], tc_[0], tc_[1],
                                            tc_[2], M, N, K, stages, ring_bytes, act, dev_status)
                  : narrow ? launch_dependent(linear_rows_kernel<256>, grid, dim3(192), (size_t)smem, s, ta, tw[0], tw[1], tw[2], tc_[0], tc_[1],
                                            tc_[2], M, N, K, stages, ring_bytes, act, dev_status)
                         : launch_dependent(linear_rows_kernel<320>, grid, dim3(192), (size_t)smem, s, ta, tw[0], tw[1], tw[2], tc_[0], tc_[1],
                                            tc_[2], M, N, K, stages, ring_bytes, act, dev_status);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace toma
