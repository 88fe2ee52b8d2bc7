// Merge X_m = A~ X (Sec. 4.2.1) and unmerge A~^T X' (Sec. 4.2.2) per tile on the sm_100a
// tensor cores: bf16 tokens, weights as a hi + lo pair of bf16 planes (two MMAs per step, ~16
// mantissa bits), fp32 accumulation in tensor memory.
//
// Both are computed transposed, with 128 feature channels on the MMA M dimension:
//   merge:    X_m^T [ch x D_loc] = X^T  [ch x N_loc] * A~^T [N_loc x D_loc]
//   unmerge:  Y^T   [ch x N_loc] = X'^T [ch x D_loc] * A~   [D_loc x N_loc]
// so the one stored weight layout A~^T [N_loc][D_loc] is the B operand of both (MN-major for the
// merge, K-major for the unmerge) and the token tensors are MN-major A operands that TMA fetches
// straight from their row-major [token][channel] storage: a spatial tile is one 4-D box of the
// (channel, x, y, batch) view of X, so no gather/reshape pass exists.
// One CTA = one (tile, 128-channel chunk, block of <= 256 output columns); warp 0 TMA, warp 1
// MMA, warps 2..5 epilogue (one thread per channel).
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kKC = 64;           // contraction elements per pipeline stage
constexpr int kSlab = kKC * 128;  // bytes of a 64-row x 128-byte slab
constexpr int kMaxCols = 256;     // output columns (MMA N) per merge CTA
constexpr int kUnmergeTok = 128;  // tokens per unmerge CTA: small enough that two CTAs share an SM

struct PipeBars {
  uint64_t full[4], empty[4], done;
  uint64_t epi;  // the four epilogue warps have staged their part of the output tile
  uint32_t tmem_base;
  int abort_flag;
};

struct LinParams {
  int P, tiles_x, th, tw, W, Nloc, Dloc, d, n_all, Lm;
  int stages;  // pipeline depth
  int dest_block;  // merge: destinations (MMA N before padding) per CTA, at most kMaxCols
  int out_rows;  // rows of one 64-channel slab of the staged output tile (= the output tensor map's box)
  uint32_t* zero;  // merge only: words cleared on the side (the attention kernel's tickets)
  int zero_words;
};

__device__ __forceinline__ uint32_t tmem_cols_for(int n) { return n > 128 ? 256u : n > 64 ? 128u : 64u; }

__device__ __forceinline__ void pipe_init(PipeBars* bar, int stages) {
  for (int s = 0; s < stages; ++s) {
    mbar_init(&bar->full[s], 1);
    mbar_init(&bar->empty[s], 1);
  }
  mbar_init(&bar->done, 1);
  mbar_init(&bar->epi, 4);
  bar->abort_flag = 0;
  mbar_fence_init();
}

// Epilogue shared by both kernels.  Thread = channel `cl` (0..127) of the CTA's chunk, holding in
// tensor memory one fp32 per output row.  The tile is staged in shared memory as two 64-channel
// slabs of [rows][128 B], 128-byte swizzled, i.e. the layout of the output tensor map's box, and
// leaves with one TMA store per slab (whole lines, asynchronous) issued by `store`.
template <typename Store>
__device__ __forceinline__ void stage_and_store(uint8_t* so, PipeBars* bar, uint32_t taddr, int cl, int n_rows, int slab_rows,
                                                uint32_t* dev_status, Store store) {
  uint8_t* mine = so + (cl >> 6) * slab_rows * 128 + (cl & 7) * 2;
  const int chunk = (cl & 63) >> 3;
  for (int i0 = 0; i0 < n_rows; i0 += 32) {
    uint32_t r[32];
    tmem_ld32(taddr + i0, r);
    tmem_wait_ld();
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const int row = i0 + e;
      if (row < n_rows)
        *reinterpret_cast<__nv_bfloat16*>(mine + row * 128 + ((chunk ^ (row & 7)) << 4)) = __float2bfloat16_rn(__uint_as_float(r[e]));
    }
  }
  fence_proxy_async();  // the staged tile is read by the TMA engine
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(&bar->epi);
  if (cl == 0 && mbar_wait(&bar->epi, 0, dev_status, &bar->abort_flag)) {
    store();
    tma_store_commit();
    tma_store_wait_read();  // shared memory must outlive the engine's reads
  }
}

// ------------------------------------------------------------------------------------------------
// merge: grid (tile, channel chunk, destination block); K loop over the tile's tokens.
// ------------------------------------------------------------------------------------------------
// kBlocked: the destinations of a region are split into blocks of p.dest_block (global merge); otherwise a
// region's destinations (<= kMaxCols) belong to one CTA and the block size is a compile-time constant.
template <bool kBlocked>
__global__ void __launch_bounds__(192, 1)
merge_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                const __grid_constant__ CUtensorMap tm_o, const LinParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int batch = blockIdx.x, c0 = blockIdx.y * 128, i_base = blockIdx.z * (kBlocked ? p.dest_block : kMaxCols);
  const int n_dest = min(kBlocked ? p.dest_block : kMaxCols, p.Dloc - i_base);  // destinations this CTA produces
  const int slabs = (n_dest + 63) / 64;               // 64-destination slabs per weight plane
  const int n_mma = slabs * 64;                       // MMA N (zero padded by TMA)
  const int stage_bytes = (2 + 2 * slabs) * kSlab;
  PipeBars* bar = reinterpret_cast<PipeBars*>(smem + p.stages * stage_bytes);
  const int b = batch / p.P, tile = batch - b * p.P;
  const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
  const int rows_per_chunk = kKC / p.tw;
  const int nk = p.Nloc / kKC;
  const uint32_t ncols = tmem_cols_for(n_mma);

  if (threadIdx.x == 0) {
    pipe_init(bar, p.stages);
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_w);
    prefetch_tmap(&tm_o);
  }
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  if (warp == 1) tmem_alloc(&bar->tmem_base, ncols);
  if (p.zero_words > 0) {
    const int cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
    const int n_thr = gridDim.x * gridDim.y * gridDim.z * blockDim.x;
    for (int i = cta * blockDim.x + threadIdx.x; i < p.zero_words; i += n_thr) p.zero[i] = 0u;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 0) {
    if (elect_one()) {
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (k >= p.stages && !mbar_wait(&bar->empty[s], ((k / p.stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sx = smem + s * stage_bytes;
        uint8_t* sw = sx + 2 * kSlab;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        for (int c = 0; c < 2; ++c)
          tma_load_4d(sx + c * kSlab, &tm_x, &bar->full[s], c0 + c * 64, tx * p.tw, ty * p.th + k * rows_per_chunk, b);
        for (int pl = 0; pl < 2; ++pl)
          for (int c = 0; c < slabs; ++c)
            tma_load_3d(sw + (pl * slabs + c) * kSlab, &tm_w, &bar->full[s], i_base + c * 64, k * kKC, 2 * batch + pl);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, true, true, 128, n_mma);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (!mbar_wait(&bar->full[s], (k / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t xa = smem_u32(smem + s * stage_bytes), wa = xa + 2 * kSlab;
#pragma unroll
        for (int kk = 0; kk < kKC / 16; ++kk) {  // 16 tokens per MMA: 16 rows of 128 B in every slab
          const uint64_t xd = smem_desc_sw128(xa + kk * 2048, kSlab, 1024);
          mma_ss(tmem, xd, smem_desc_sw128(wa + kk * 2048, kSlab, 1024), idesc, k > 0 || kk > 0);
          mma_ss(tmem, xd, smem_desc_sw128(wa + slabs * kSlab + kk * 2048, kSlab, 1024), idesc, true);
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3, cl = quarter * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    if (mbar_wait(&bar->done, 0, dev_status, abort_flag)) {  // every load has been consumed: the stages are free
      tc_fence_after();
      stage_and_store(smem, bar, taddr, cl, n_dest, p.out_rows, dev_status, [&] {
        for (int c = 0; c < 2; ++c)
          if (c0 + c * 64 < p.d) tma_store_4d(&tm_o, smem + c * p.out_rows * 128, c0 + c * 64, i_base, tile, b);
      });
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

// ------------------------------------------------------------------------------------------------
// merge, persistent form: for launches of many more (tile, channel chunk) items than the SMs hold at once.
// One CTA per SM takes items blockIdx.x, blockIdx.x + gridDim.x, ... (consecutive CTAs work on chunks of the same
// tile, so the tile's weights are L2 hits for all but one of them).  The TMA ring runs on across items; two
// accumulators in tensor memory alternate, so that an item's epilogue (tensor memory -> staging tile in shared
// memory -> TMA store) runs under the next item's loads and MMAs, and the prologue, the cold first fetch and
// the tail of a CTA are paid once per SM instead of once per item.
// ------------------------------------------------------------------------------------------------
struct PersistBars {
  uint64_t full[4], empty[4];
  uint64_t acc_full[2], acc_empty[2];  // accumulator complete / read out by the four epilogue warps
  uint64_t staged, stored;             // the staging tile is written (4 warps) / the TMA store has read it
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(192, 1)
merge_persistent_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                        const __grid_constant__ CUtensorMap tm_o, const LinParams p, int n_items, int n_chunks,
                        uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_dest = p.Dloc;                          // <= kMaxCols: one CTA produces all of a tile's destinations
  const int slabs = (n_dest + 63) / 64, n_mma = slabs * 64;
  const int stage_bytes = (2 + 2 * slabs) * kSlab;
  uint8_t* so = smem + p.stages * stage_bytes;        // staging tile: two 64-channel slabs of [out_rows][128 B]
  PersistBars* bar = reinterpret_cast<PersistBars*>(so + 2 * p.out_rows * 128);
  const int rows_per_chunk = kKC / p.tw;
  const int nk = p.Nloc / kKC;
  const uint32_t acc_cols = tmem_cols_for(n_mma);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&bar->acc_full[a], 1);
      mbar_init(&bar->acc_empty[a], 4);
    }
    mbar_init(&bar->staged, 4);
    mbar_init(&bar->stored, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_w);
    prefetch_tmap(&tm_o);
  }
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  if (warp == 1) tmem_alloc(&bar->tmem_base, 2 * acc_cols);
  if (p.zero_words > 0) {
    const int n_thr = gridDim.x * blockDim.x;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < p.zero_words; i += n_thr) p.zero[i] = 0u;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 0) {
    if (elect_one()) {
      int kc = 0;  // k-steps issued so far, over all items: ring slot and phase follow it
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const int batch = item / n_chunks, c0 = (item - batch * n_chunks) * 128;
        const int b = batch / p.P, tile = batch - b * p.P;
        const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
        for (int k = 0; k < nk; ++k, ++kc) {
          const int s = kc % p.stages;
          if (kc >= p.stages && !mbar_wait(&bar->empty[s], ((kc / p.stages) - 1) & 1, dev_status, abort_flag)) { ok = false; break; }
          uint8_t* sx = smem + s * stage_bytes;
          uint8_t* sw = sx + 2 * kSlab;
          mbar_expect_tx(&bar->full[s], stage_bytes);
          for (int c = 0; c < 2; ++c)
            tma_load_4d(sx + c * kSlab, &tm_x, &bar->full[s], c0 + c * 64, tx * p.tw, ty * p.th + k * rows_per_chunk, b);
          for (int pl = 0; pl < 2; ++pl)
            for (int c = 0; c < slabs; ++c)
              tma_load_3d(sw + (pl * slabs + c) * kSlab, &tm_w, &bar->full[s], c * 64, k * kKC, 2 * batch + pl);
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, true, true, 128, n_mma);
      int kc = 0, n = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
        const int a = n & 1;
        if (n >= 2 && !mbar_wait(&bar->acc_empty[a], ((n >> 1) - 1) & 1, dev_status, abort_flag)) break;
        tc_fence_after();
        const uint32_t t_acc = tmem + a * acc_cols;
        bool ok = true;
        for (int k = 0; k < nk; ++k, ++kc) {
          const int s = kc % p.stages;
          if (!mbar_wait(&bar->full[s], (kc / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t xa = smem_u32(smem + s * stage_bytes), wa = xa + 2 * kSlab;
#pragma unroll
          for (int kk = 0; kk < kKC / 16; ++kk) {
            const uint64_t xd = smem_desc_sw128(xa + kk * 2048, kSlab, 1024);
            mma_ss(t_acc, xd, smem_desc_sw128(wa + kk * 2048, kSlab, 1024), idesc, k > 0 || kk > 0);
            mma_ss(t_acc, xd, smem_desc_sw128(wa + slabs * kSlab + kk * 2048, kSlab, 1024), idesc, true);
          }
          mma_commit(&bar->empty[s]);
        }
        if (!ok) break;
        mma_commit(&bar->acc_full[a]);
      }
    }
  } else {
    const int quarter = warp & 3, cl = quarter * 32 + lane;  // channel of the chunk = tensor-memory lane
    uint8_t* mine = so + (cl >> 6) * p.out_rows * 128 + (cl & 7) * 2;
    const int chunk = (cl & 63) >> 3;
    int n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const int a = n & 1;
      const int batch = item / n_chunks, c0 = (item - batch * n_chunks) * 128;
      const int b = batch / p.P, tile = batch - b * p.P;
      // the accumulator is complete, and the previous item's store has read the staging tile that is written
      // again below; one answer per warp (the tensor-memory loads are warp-wide operations)
      const bool go = mbar_wait(&bar->acc_full[a], (n >> 1) & 1, dev_status, abort_flag) &&
                      (n == 0 || mbar_wait(&bar->stored, (n - 1) & 1, dev_status, abort_flag));
      if (!__all_sync(0xffffffffu, go)) break;
      tc_fence_after();
      const uint32_t taddr = tmem + a * acc_cols + ((uint32_t)(quarter * 32) << 16);
      for (int i0 = 0; i0 < n_dest; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int row = i0 + e;
          if (row < n_dest)
            *reinterpret_cast<__nv_bfloat16*>(mine + row * 128 + ((chunk ^ (row & 7)) << 4)) = __float2bfloat16_rn(__uint_as_float(r[e]));
        }
      }
      tc_fence_before();
      fence_proxy_async();  // the staged tile is read by the TMA engine
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bar->acc_empty[a]);  // the accumulator may be overwritten by the item after next
        mbar_arrive(&bar->staged);
      }
      if (cl == 0 && mbar_wait(&bar->staged, n & 1, dev_status, abort_flag)) {  // a wait that ran out ends the loop at its top
        for (int c = 0; c < 2; ++c)
          if (c0 + c * 64 < p.d) tma_store_4d(&tm_o, so + c * p.out_rows * 128, c0 + c * 64, 0, tile, b);
        tma_store_commit();
        tma_store_wait_read();  // shared memory must outlive the engine's reads
        mbar_arrive(&bar->stored);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * acc_cols);
  }
}

// ------------------------------------------------------------------------------------------------
// unmerge: grid (tile, channel chunk, token block); K loop over the tile's destinations.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(192, 1)
unmerge_tc_kernel(const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_w,
                  const __grid_constant__ CUtensorMap tm_o, const LinParams p, int n_tok, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int w_plane = n_tok * 128;  // bytes of one [n_tok tokens][64 destinations] weight block
  const int stage_bytes = 2 * kSlab + 2 * w_plane;
  PipeBars* bar = reinterpret_cast<PipeBars*>(smem + p.stages * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int batch = blockIdx.x, c0 = blockIdx.y * 128, t0 = blockIdx.z * n_tok;
  const int b = batch / p.P, tile = batch - b * p.P;
  const int nk = (p.Dloc + kKC - 1) / kKC;
  const uint32_t ncols = tmem_cols_for(n_tok);

  if (threadIdx.x == 0) {
    pipe_init(bar, p.stages);
    prefetch_tmap(&tm_y);
    prefetch_tmap(&tm_w);
    prefetch_tmap(&tm_o);
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
        const int s = k % p.stages;
        if (k >= p.stages && !mbar_wait(&bar->empty[s], ((k / p.stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sy = smem + s * stage_bytes;
        uint8_t* sw = sy + 2 * kSlab;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        for (int c = 0; c < 2; ++c)
          tma_load_3d(sy + c * kSlab, &tm_y, &bar->full[s], c0 + c * 64, tile * p.Dloc + k * kKC, b);
        for (int pl = 0; pl < 2; ++pl) tma_load_3d(sw + pl * w_plane, &tm_w, &bar->full[s], k * kKC, t0, 2 * batch + pl);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, true, false, 128, n_tok);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (!mbar_wait(&bar->full[s], (k / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ya = smem_u32(smem + s * stage_bytes), wa = ya + 2 * kSlab;
        const int ksteps = min(kKC, p.Dloc - k * kKC + 15) / 16;  // 16 destinations per MMA
        for (int kk = 0; kk < ksteps; ++kk) {
          const uint64_t yd = smem_desc_sw128(ya + kk * 2048, kSlab, 1024);
          mma_ss(tmem, yd, smem_desc_sw128(wa + kk * 32, 16, 1024), idesc, k > 0 || kk > 0);
          mma_ss(tmem, yd, smem_desc_sw128(wa + w_plane + kk * 32, 16, 1024), idesc, true);
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3, cl = quarter * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    if (mbar_wait(&bar->done, 0, dev_status, abort_flag)) {
      tc_fence_after();
      // rows of the staged tile = the CTA's token slots in tile order = the (x, y) box of the output map
      const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
      stage_and_store(smem, bar, taddr, cl, n_tok, n_tok, dev_status, [&] {
        for (int c = 0; c < 2; ++c)
          if (c0 + c * 64 < p.d)
            tma_store_4d(&tm_o, smem + c * n_tok * 128, c0 + c * 64, tx * p.tw, ty * p.th + t0 / p.tw, b);
      });
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

// ------------------------------------------------------------------------------------------------
// unmerge for regions with many destinations (global merge), tokens on M:
//   Y [tok x ch] = A~^T [tok x D] * X' [D x ch]
// one CTA = (128 tokens, block of up to 320 channels).  The stored weights are the K-major A operand
// as they are, the attended rows an MN-major B operand (two MMAs along N: at most 192 + 128 channels).
// Against channels on M (128 x 128 tiles) a k-step moves 72 KB for 10.5 MFLOP instead of 48 KB for
// 4.2 MFLOP, the weights are read twice instead of five times, and the 128 CTAs of the 64x64-token
// case fit the SMs in one wave with a three-stage pipeline; each thread then owns a token row, which it
// stages in shared memory (the pipeline's stages, free by then) as 64-channel slabs in the layout of the
// output tensor map's box: the CTA's 128 tokens are whole tile rows, one TMA store per slab.
// ------------------------------------------------------------------------------------------------
constexpr int kRowsChBlock = 320;  // channels per CTA (five 64-channel slabs)

__global__ void __launch_bounds__(192, 1)
unmerge_rows_kernel(const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_o, const LinParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks_per_tile = p.Nloc / 128;
  const int batch = blockIdx.x / blocks_per_tile, t0 = (blockIdx.x - batch * blocks_per_tile) * 128;
  const int b = batch / p.P, tile = batch - b * p.P;
  const int c0 = blockIdx.y * kRowsChBlock;
  const int n_ch = min(kRowsChBlock, p.d - c0);   // channels of this CTA (multiple of 8)
  const int slabs = (n_ch + 63) / 64;             // 64-channel slabs of the B operand
  const int n_a = min(slabs, 3) * 64;             // MMA N of the first accumulator (<= 192)
  const int n_b = (slabs - min(slabs, 3)) * 64;   // and of the second (0, 64 or 128)
  const int w_plane = 128 * 128;                  // [128 tokens][64 destinations] of one plane
  const int stage_bytes = 2 * w_plane + slabs * kSlab;
  PipeBars* bar = reinterpret_cast<PipeBars*>(smem + p.stages * stage_bytes);
  const int nk = (p.Dloc + kKC - 1) / kKC;
  constexpr uint32_t ncols = 512;

  if (threadIdx.x == 0) {
    pipe_init(bar, p.stages);
    prefetch_tmap(&tm_y);
    prefetch_tmap(&tm_w);
    prefetch_tmap(&tm_o);
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
        const int s = k % p.stages;
        if (k >= p.stages && !mbar_wait(&bar->empty[s], ((k / p.stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sw = smem + s * stage_bytes;
        uint8_t* sy = sw + 2 * w_plane;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        for (int pl = 0; pl < 2; ++pl) tma_load_3d(sw + pl * w_plane, &tm_w, &bar->full[s], k * kKC, t0, 2 * batch + pl);
        for (int c = 0; c < slabs; ++c)
          tma_load_3d(sy + c * kSlab, &tm_y, &bar->full[s], c0 + c * 64, tile * p.Dloc + k * kKC, b);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc_a = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_a);
      const uint32_t idesc_b = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_b > 0 ? n_b : 64);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (!mbar_wait(&bar->full[s], (k / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t wa = smem_u32(smem + s * stage_bytes), ya = wa + 2 * w_plane;
        const int ksteps = min(kKC, p.Dloc - k * kKC + 15) / 16;  // 16 destinations per MMA
        for (int kk = 0; kk < ksteps; ++kk) {
          const uint64_t yd_a = smem_desc_sw128(ya + kk * 2048, kSlab, 1024);
          const uint64_t yd_b = smem_desc_sw128(ya + 3 * kSlab + kk * 2048, kSlab, 1024);
          for (int pl = 0; pl < 2; ++pl) {
            const uint64_t wd = smem_desc_sw128(wa + pl * w_plane + kk * 32, 16, 1024);
            const bool acc = k > 0 || kk > 0 || pl > 0;
            mma_ss(tmem, wd, yd_a, idesc_a, acc);
            if (n_b > 0) mma_ss(tmem + 192, wd, yd_b, idesc_b, acc);
          }
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3, row = quarter * 32 + lane;  // token slot t0 + row = tensor-memory lane
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    if (mbar_wait(&bar->done, 0, dev_status, abort_flag)) {
      tc_fence_after();
      // every load has been consumed: slab c of the output, [128 tokens][128 B] swizzled, goes to smem + c * 16 KB
      for (int c = 0; c < n_ch; c += 32) {  // accumulator column = channel (the second accumulator starts at 192)
        uint32_t r[32];
        tmem_ld32(taddr + c, r);
        tmem_wait_ld();
        uint8_t* slab = smem + (c >> 6) * (128 * 128);
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          if (c + e < n_ch) {
            __align__(16) __nv_bfloat162 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              q[u] = __floats2bfloat162_rn(__uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1]));
            *reinterpret_cast<uint4*>(slab + sw128_offset(row, ((c & 63) + e) >> 3)) = *reinterpret_cast<const uint4*>(q);
          }
        }
      }
      fence_proxy_async();  // the staged rows are read by the TMA engine
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->epi);
      if (row == 0 && mbar_wait(&bar->epi, 0, dev_status, abort_flag)) {
        const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
        for (int c = 0; c < slabs; ++c)  // a slab cut short by the channel count is clipped by the store
          tma_store_4d(&tm_o, smem + c * (128 * 128), c0 + c * 64, tx * p.tw, ty * p.th + t0 / p.tw, b);
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

// ------------------------------------------------------------------------------------------------
// unmerge with tokens on M, persistent form: for launches of many more (tile, 128-token block, channel block)
// items than there are SMs.  One CTA per SM walks its items; the ring holds the next item's operands while the
// current one is multiplied, the output tile has a staging area of its own, and an item's TMA store runs
// under the next item's MMAs.  One accumulator set (up to 320 columns of tensor memory): the next item's MMAs
// wait only until the epilogue warps have read the accumulators out.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(192, 1)
unmerge_rows_persistent_kernel(const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_w,
                               const __grid_constant__ CUtensorMap tm_o, const LinParams p, int n_items, int ch_blocks,
                               uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks_per_tile = p.Nloc / 128;
  const int max_slabs = ((p.d < kRowsChBlock ? p.d : kRowsChBlock) + 63) / 64;
  const int w_plane = 128 * 128;  // [128 tokens][64 destinations] of one plane
  const int stage_bytes = 2 * w_plane + max_slabs * kSlab;
  uint8_t* so = smem + p.stages * stage_bytes;  // staging: max_slabs slabs of [128 tokens][128 B]
  PersistBars* bar = reinterpret_cast<PersistBars*>(so + max_slabs * (128 * 128));
  const int nk = (p.Dloc + kKC - 1) / kKC;
  constexpr uint32_t ncols = 512;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->acc_full[0], 1);
    mbar_init(&bar->acc_empty[0], 4);
    mbar_init(&bar->staged, 4);
    mbar_init(&bar->stored, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_y);
    prefetch_tmap(&tm_w);
    prefetch_tmap(&tm_o);
  }
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  if (warp == 1) tmem_alloc(&bar->tmem_base, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;
  // item -> (tile of the batch, 128-token block, channel block); channel blocks of one token block are neighbours,
  // so that concurrently running CTAs share its weights in L2
  auto decode = [&](int item, int& batch, int& t0, int& c0) {
    const int cb = item % ch_blocks, tb = item / ch_blocks;
    batch = tb / blocks_per_tile;
    t0 = (tb - batch * blocks_per_tile) * 128;
    c0 = cb * kRowsChBlock;
  };

  if (warp == 0) {
    if (elect_one()) {
      int kc = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        int batch, t0, c0;
        decode(item, batch, t0, c0);
        const int b = batch / p.P, tile = batch - b * p.P;
        const int slabs = (min(kRowsChBlock, p.d - c0) + 63) / 64;
        for (int k = 0; k < nk; ++k, ++kc) {
          const int s = kc % p.stages;
          if (kc >= p.stages && !mbar_wait(&bar->empty[s], ((kc / p.stages) - 1) & 1, dev_status, abort_flag)) { ok = false; break; }
          uint8_t* sw = smem + s * stage_bytes;
          uint8_t* sy = sw + 2 * w_plane;
          mbar_expect_tx(&bar->full[s], 2 * w_plane + slabs * kSlab);
          for (int pl = 0; pl < 2; ++pl) tma_load_3d(sw + pl * w_plane, &tm_w, &bar->full[s], k * kKC, t0, 2 * batch + pl);
          for (int c = 0; c < slabs; ++c)
            tma_load_3d(sy + c * kSlab, &tm_y, &bar->full[s], c0 + c * 64, tile * p.Dloc + k * kKC, b);
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      int kc = 0, n = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++n) {
        int batch, t0, c0;
        decode(item, batch, t0, c0);
        const int slabs = (min(kRowsChBlock, p.d - c0) + 63) / 64;
        const int n_a = min(slabs, 3) * 64, n_b = (slabs - min(slabs, 3)) * 64;
        const uint32_t idesc_a = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_a);
        const uint32_t idesc_b = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, n_b > 0 ? n_b : 64);
        // the epilogue warps have read the previous item's accumulators
        if (n >= 1 && !mbar_wait(&bar->acc_empty[0], (n - 1) & 1, dev_status, abort_flag)) break;
        tc_fence_after();
        for (int k = 0; k < nk; ++k, ++kc) {
          const int s = kc % p.stages;
          if (!mbar_wait(&bar->full[s], (kc / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t wa = smem_u32(smem + s * stage_bytes), ya = wa + 2 * w_plane;
          const int ksteps = min(kKC, p.Dloc - k * kKC + 15) / 16;  // 16 destinations per MMA
          for (int kk = 0; kk < ksteps; ++kk) {
            const uint64_t yd_a = smem_desc_sw128(ya + kk * 2048, kSlab, 1024);
            const uint64_t yd_b = smem_desc_sw128(ya + 3 * kSlab + kk * 2048, kSlab, 1024);
            for (int pl = 0; pl < 2; ++pl) {
              const uint64_t wd = smem_desc_sw128(wa + pl * w_plane + kk * 32, 16, 1024);
              const bool acc = k > 0 || kk > 0 || pl > 0;
              mma_ss(tmem, wd, yd_a, idesc_a, acc);
              if (n_b > 0) mma_ss(tmem + 192, wd, yd_b, idesc_b, acc);
            }
          }
          mma_commit(&bar->empty[s]);
        }
        if (ok) mma_commit(&bar->acc_full[0]);
      }
    }
  } else {
    const int quarter = warp & 3, row = quarter * 32 + lane;  // token slot t0 + row = tensor-memory lane
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    int n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      int batch, t0, c0;
      decode(item, batch, t0, c0);
      const int b = batch / p.P, tile = batch - b * p.P;
      const int n_ch = min(kRowsChBlock, p.d - c0), slabs = (n_ch + 63) / 64;
      // the accumulators are complete, and the previous item's store has read the staging area; one answer per
      // warp (the tensor-memory loads are warp-wide operations)
      const bool go = mbar_wait(&bar->acc_full[0], n & 1, dev_status, abort_flag) &&
                      (n == 0 || mbar_wait(&bar->stored, (n - 1) & 1, dev_status, abort_flag));
      if (!__all_sync(0xffffffffu, go)) break;
      tc_fence_after();
      for (int c = 0; c < n_ch; c += 32) {  // accumulator column = channel (the second accumulator starts at 192)
        uint32_t r[32];
        tmem_ld32(taddr + c, r);
        tmem_wait_ld();
        uint8_t* slab = so + (c >> 6) * (128 * 128);
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          if (c + e < n_ch) {
            __align__(16) __nv_bfloat162 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              q[u] = __floats2bfloat162_rn(__uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1]));
            *reinterpret_cast<uint4*>(slab + sw128_offset(row, ((c & 63) + e) >> 3)) = *reinterpret_cast<const uint4*>(q);
          }
        }
      }
      tc_fence_before();
      fence_proxy_async();  // the staged rows are read by the TMA engine
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bar->acc_empty[0]);  // the next item's products may overwrite the accumulators
        mbar_arrive(&bar->staged);
      }
      if (row == 0 && mbar_wait(&bar->staged, n & 1, dev_status, abort_flag)) {  // a wait that ran out ends the loop at its top
        const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
        for (int c = 0; c < slabs; ++c)  // a slab cut short by the channel count is clipped by the store
          tma_store_4d(&tm_o, so + c * (128 * 128), c0 + c * 64, tx * p.tw, ty * p.th + t0 / p.tw, b);
        tma_store_commit();
        tma_store_wait_read();  // shared memory must outlive the engine's reads
        mbar_arrive(&bar->stored);
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

LinParams make_params(const Geom& g) {
  LinParams p;
  p.P = g.P; p.tiles_x = g.tiles_x; p.th = g.th; p.tw = g.tw; p.W = g.W; p.Nloc = g.Nloc; p.Dloc = g.Dloc;
  p.d = g.d; p.n_all = (int)g.tokens_all(); p.Lm = g.Lm; p.stages = 2;
  p.zero = nullptr; p.zero_words = 0; p.out_rows = 0; p.dest_block = 0;
  return p;
}

// Weight planes as a 3-D tensor (destination, token, plane): plane 2*tile is hi, 2*tile + 1 is lo.
bool encode_w(const Geom& g, const void* w, CUtensorMap* tm, uint32_t box_tokens) {
  const uint64_t dims[3] = {(uint64_t)g.Dloc, (uint64_t)g.Nloc, (uint64_t)g.B * g.P * 2};
  const uint64_t strides[2] = {(uint64_t)g.Dloc * 2, (uint64_t)g.Nloc * g.Dloc * 2};
  const uint32_t box[3] = {64, box_tokens, 1};
  return encode_tmap_16bit(tm, w, 3, dims, strides, box);
}

}  // namespace

// Shapes the tensor-core merge / unmerge cover; everything else runs on the FFMA kernels.
bool linear_tc_supported(const Geom& g) {
  if (g.f32) return false;
  if (g.tw > 64 || (64 % g.tw) != 0 || (g.th % (64 / g.tw)) != 0) return false;  // 64 tokens = whole tile rows
  // The unmerge multiplies destinations 16 at a time out of rows addressed as one (rows, channels)
  // sheet of the merged tensor: with D_loc a multiple of 16 a step never touches a row of the next tile.
  if (g.Nloc % 64 != 0 || g.Dloc % 16 != 0) return false;
  if (g.Nloc > kUnmergeTok && g.Nloc % kUnmergeTok != 0) return false;  // unmerge token blocks
  return true;
}

cudaError_t launch_merge_tc(const Geom& g, const void* w, const void* x, void* xm, void* zero, size_t zero_bytes,
                            uint32_t* dev_status, cudaStream_t s) {
  CUtensorMap tx, tw;
  const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t strides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t box[4] = {64, (uint32_t)g.tw, (uint32_t)(64 / g.tw), 1};
  if (!encode_tmap_16bit(&tx, x, 4, dims, strides, box) || !encode_w(g, w, &tw, 64)) return cudaErrorInvalidValue;
  LinParams p = make_params(g);
  // merged rows as (channel, destination, tile, batch): a store that runs past a tile's D_loc rows is clipped
  CUtensorMap to;
  // Destinations per CTA.  A tile's destinations normally fit one CTA (<= 256).  When they do not (global
  // merge) the launch is bound by how many bytes the SMs keep in flight, so the block size is the
  // one that gives every SM a CTA with the deepest pipeline its shared memory holds: the largest multiple
  // of 16 whose CTA count does not exceed the SM count (a few CTAs more would double the run time).
  p.dest_block = g.Dloc < kMaxCols ? g.Dloc : kMaxCols;
  if (g.Dloc > kMaxCols) {
    const int sms = sm_count();
    const int per_block = g.B * g.P * ((g.d + 127) / 128);  // CTAs per destination block
    for (int nb = (g.Dloc + kMaxCols - 1) / kMaxCols; nb * per_block <= sms; ++nb) {
      const int cand = (((g.Dloc + nb - 1) / nb) + 15) & ~15;
      if (cand >= 64) p.dest_block = cand;
    }
  }
  p.out_rows = p.dest_block;
  const uint64_t odims[4] = {(uint64_t)g.d, (uint64_t)g.Dloc, (uint64_t)g.P, (uint64_t)g.B};
  const uint64_t ostrides[3] = {(uint64_t)g.d * 2, (uint64_t)g.Dloc * g.d * 2, (uint64_t)g.Lm * g.d * 2};
  const uint32_t obox[4] = {64, (uint32_t)p.out_rows, 1, 1};
  if (!encode_tmap_16bit(&to, xm, 4, odims, ostrides, obox)) return cudaErrorInvalidValue;
  const int slabs = (p.dest_block + 63) / 64;
  const int stage_bytes = (2 + 2 * slabs) * kSlab;
  p.zero = (uint32_t*)zero;
  p.zero_words = (int)(zero_bytes / 4);
  p.stages = 2;  // two stages keep a CTA below ~100 KB so that two or three CTAs share an SM and hide each other's latencies
  if (g.Dloc > kMaxCols) {  // one CTA per SM anyway: as deep as shared memory allows
    p.stages = (198 * 1024) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages < 2 ? 2 : p.stages;
  }
  if (p.stages > g.Nloc / kKC) p.stages = g.Nloc / kKC;
  const int smem = 1024 + p.stages * stage_bytes + 256;
  dim3 grid(g.B * g.P, (g.d + 127) / 128, (g.Dloc + p.dest_block - 1) / p.dest_block);
  cudaError_t e;
  const int n_chunks = (g.d + 127) / 128, n_items = g.B * g.P * n_chunks;
  if (g.Dloc <= kMaxCols && n_items > 2 * sm_count()) {
    // more items than the SMs hold at once: one CTA per SM walks them with the ring and two accumulators kept busy
    const int staging = 2 * p.out_rows * 128;
    p.stages = (227 * 1024 - 1024 - 512 - staging) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages;
    if (p.stages >= 2) {
      const int smem_p = 1024 + p.stages * stage_bytes + staging + 512;
      static std::atomic<unsigned long long> raised_p{0};
      e = raise_dynamic_smem(merge_persistent_kernel, 227 * 1024, raised_p);
      if (e != cudaSuccess) return e;
      const int ctas = n_items < sm_count() ? n_items : sm_count();
      e = launch_dependent(merge_persistent_kernel, dim3(ctas), dim3(192), (size_t)smem_p, s, tx, tw, to, p, n_items, n_chunks, dev_status);
      count_launch();
      return e != cudaSuccess ? e : cudaGetLastError();
    }
    p.stages = 2;
  }
  if (g.Dloc > kMaxCols) {
    static std::atomic<unsigned long long> raised_b{0};
    e = raise_dynamic_smem(merge_tc_kernel<true>, 200 * 1024, raised_b);
    if (e != cudaSuccess) return e;
    e = launch_dependent(merge_tc_kernel<true>, grid, dim3(192), (size_t)smem, s, tx, tw, to, p, dev_status);
  } else {
    static std::atomic<unsigned long long> raised{0};
    e = raise_dynamic_smem(merge_tc_kernel<false>, 200 * 1024, raised);
    if (e != cudaSuccess) return e;
    e = launch_dependent(merge_tc_kernel<false>, grid, dim3(192), (size_t)smem, s, tx, tw, to, p, dev_status);
  }
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_unmerge_tc(const Geom& g, const void* w, const void* y, void* out, uint32_t* dev_status,
                              cudaStream_t s) {
  CUtensorMap ty, tw;
  const int n_tok = g.Nloc > kUnmergeTok ? kUnmergeTok : g.Nloc;
  const uint64_t dims[3] = {(uint64_t)g.d, (uint64_t)g.Lm, (uint64_t)g.B};
  const uint64_t strides[2] = {(uint64_t)g.d * 2, (uint64_t)g.Lm * g.d * 2};
  const uint32_t box[3] = {64, 64, 1};
  if (!encode_tmap_16bit(&ty, y, 3, dims, strides, box) || !encode_w(g, w, &tw, (uint32_t)n_tok))
    return cudaErrorInvalidValue;
  LinParams p = make_params(g);
  // Tokens on M when a region has many destinations, and also when that form fits the SMs in one wave while
  // the channels-on-M grid would spill into a second one (64x64 tokens: 128 CTAs against 320 on 296 slots).
  const int sms = sm_count();
  const int rows_ctas = g.B * g.P * (g.Nloc / 128) * ((g.d + kRowsChBlock - 1) / kRowsChBlock);
  const int classic_ctas = g.B * g.P * ((g.d + 127) / 128) * (g.Nloc / n_tok);
  const bool one_wave = rows_ctas <= sms && classic_ctas > 2 * sms;
  if (g.Dloc <= kMaxCols && g.Nloc % 128 == 0 && rows_ctas > sms) {
    // many more items than SMs: tokens on M, one CTA per SM walking its items
    CUtensorMap tw128, to;
    if (!encode_w(g, w, &tw128, 128)) return cudaErrorInvalidValue;
    const uint64_t odims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
    const uint64_t ostrides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
    const uint32_t obox[4] = {64, (uint32_t)g.tw, (uint32_t)(128 / g.tw), 1};
    if (!encode_tmap_16bit(&to, out, 4, odims, ostrides, obox)) return cudaErrorInvalidValue;
    const int max_slabs = ((g.d < kRowsChBlock ? g.d : kRowsChBlock) + 63) / 64;
    const int stage_bytes = 2 * 128 * 128 + max_slabs * kSlab, staging = max_slabs * 128 * 128;
    p.stages = (227 * 1024 - 1024 - 512 - staging) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages;
    if (p.stages >= 2) {
      const int smem = 1024 + p.stages * stage_bytes + staging + 512;
      static std::atomic<unsigned long long> raised_rp{0};
      if (cudaError_t e = raise_dynamic_smem(unmerge_rows_persistent_kernel, 227 * 1024, raised_rp); e != cudaSuccess) return e;
      const int ch_blocks = (g.d + kRowsChBlock - 1) / kRowsChBlock;
      cudaError_t e = launch_dependent(unmerge_rows_persistent_kernel, dim3(sms), dim3(192), (size_t)smem, s, ty, tw128, to, p, rows_ctas,
                                       ch_blocks, dev_status);
      count_launch();
      return e != cudaSuccess ? e : cudaGetLastError();
    }
  }
  if ((g.Dloc > kMaxCols || one_wave) && g.Nloc % 128 == 0) {
    CUtensorMap tw128;
    if (!encode_w(g, w, &tw128, 128)) return cudaErrorInvalidValue;
    const int slabs = ((g.d < kRowsChBlock ? g.d : kRowsChBlock) + 63) / 64;
    const int stage_bytes = 2 * 128 * 128 + slabs * kSlab;
    p.stages = (224 * 1024) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages < 2 ? 2 : p.stages;
    // never fewer than two: the stages double as the staging area of the output (slabs x 16 KB <= 2 stages)
    if (p.stages > (g.Dloc + kKC - 1) / kKC) p.stages = (g.Dloc + kKC - 1) / kKC < 2 ? 2 : (g.Dloc + kKC - 1) / kKC;
    const int smem = 1024 + p.stages * stage_bytes + 256;
    static std::atomic<unsigned long long> raised_r{0};
    if (cudaError_t e = raise_dynamic_smem(unmerge_rows_kernel, 227 * 1024, raised_r); e != cudaSuccess) return e;
    // output tokens as (channel, x, y, batch): a CTA's 128 tokens are 128 / tile_w whole tile rows
    CUtensorMap to;
    const uint64_t odims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
    const uint64_t ostrides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
    const uint32_t obox[4] = {64, (uint32_t)g.tw, (uint32_t)(128 / g.tw), 1};
    if (!encode_tmap_16bit(&to, out, 4, odims, ostrides, obox)) return cudaErrorInvalidValue;
    dim3 grid(g.B * g.P * (g.Nloc / 128), (g.d + kRowsChBlock - 1) / kRowsChBlock);
    cudaError_t e = launch_dependent(unmerge_rows_kernel, grid, dim3(192), (size_t)smem, s, ty, tw128, to, p, dev_status);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  // output tokens as (channel, x, y, batch): a CTA's token block is n_tok / tile_w whole tile rows
  CUtensorMap to;
  const uint64_t odims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t ostrides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t obox[4] = {64, (uint32_t)g.tw, (uint32_t)(n_tok / g.tw), 1};
  if (!encode_tmap_16bit(&to, out, 4, odims, ostrides, obox)) return cudaErrorInvalidValue;
  const int stage_bytes = 2 * kSlab + 2 * n_tok * 128;
  p.stages = 2;
  if (p.stages > (g.Dloc + kKC - 1) / kKC) p.stages = (g.Dloc + kKC - 1) / kKC;
  const int smem = 1024 + p.stages * stage_bytes + 256;
  static std::atomic<unsigned long long> raised{0};
  cudaError_t e = raise_dynamic_smem(unmerge_tc_kernel, 200 * 1024, raised);
  if (e != cudaSuccess) return e;
  dim3 grid(g.B * g.P, (g.d + 127) / 128, g.Nloc / n_tok);
  e = launch_dependent(unmerge_tc_kernel, grid, dim3(192), (size_t)smem, s, ty, tw, to, p, n_tok, dev_status);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace toma
