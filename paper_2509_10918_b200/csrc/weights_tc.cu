// Merge weights (Sec. 4.2.1) on the tensor cores, bf16 mode.
//
//   1. gather_dest_kernel: copies the D_loc selected tokens of every tile into a dense
//      [tile][D_loc][d] buffer so that TMA can feed them as an MMA operand.
//   2. weights_logits_kernel: L^T [source k][destination i] = <X_k, X_idx_i> with 128 source
//      tokens on the MMA M dimension, so each epilogue thread owns one source token and the softmax
//      over the DESTINATION axis (a source token's shares sum to 1) is a private register
//      reduction over its tensor-memory row.  Writes the shares A_ik (fp32) and, per 128-source
//      block, the partial row sums sum_k A_ik.
//   3. weights_normalise_kernel: A~_ik = A_ik / sum_k' A_ik' with the partial sums added in a
//      fixed order, stored as A~^T [N_loc][D_loc] split into a hi and a lo bf16 plane.
// Tiles of at most 256 tokens and 256 destinations take weights_fused_kernel instead of 2 and 3: one
// CTA per tile, the row normalisation applied in the epilogue of the logits contraction.
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kKC = 64;

struct WBars {
  uint64_t full[4], empty[4], done;
  uint64_t z_in;  // paired form: the peer CTA's row sums have arrived
  uint32_t tmem_base;
  int abort_flag;
};

struct WParams {
  int P, tiles_x, th, tw, W, Nloc, Dloc, d, n_all;
  int m_tok;    // source tokens per CTA (128, or N_loc when the tile is smaller)
  int stages;
  float scale_log2;  // log2(e) / (tau * sqrt(d))
  int d_block;  // destinations per CTA: D_loc itself, or 512 when D_loc is larger (blockIdx.z picks the block)
  int raw;      // 1: write the scaled logits (log2 domain) only; the softmax over all blocks runs afterwards
};

__global__ void __launch_bounds__(256)
gather_dest_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ idx, __nv_bfloat16* __restrict__ dg,
                   WParams p, int rows_total) {
  dependency_wait();  // launched with programmatic stream serialisation
  if (threadIdx.x == 0) release_dependents();
  const int vec_per_row = p.d / 8;  // 16-byte packets
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)rows_total * vec_per_row) return;
  const int row = (int)(e / vec_per_row), v = (int)(e - (long long)row * vec_per_row);
  const int batch = row / p.Dloc;
  const int b = batch / p.P, tile = batch - b * p.P;
  const int tok = tile_token(tile, idx[row], p.tiles_x, p.th, p.tw, p.W);
  const uint4* src = reinterpret_cast<const uint4*>(x + ((size_t)b * p.n_all + tok) * p.d) + v;
  reinterpret_cast<uint4*>(dg + (size_t)row * p.d)[v] = *src;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(192, 1)
weights_logits_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_d,
                      float* __restrict__ shares, float* __restrict__ zpart, const WParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int d_base = blockIdx.z * p.d_block;     // first destination of this CTA
  const int Dl = min(p.d_block, p.Dloc - d_base);  // its destinations
  const int n_mma = (Dl + 15) & ~15;              // MMA N: destinations padded to 16
  const int n0 = n_mma > 256 ? 256 : n_mma, n1 = n_mma - n0;
  const int a_bytes = 128 * 128;
  const int b_rows = (p.raw || Dl > 256) ? 512 : ((Dl + 7) & ~7);  // rows the swizzled operand tile spans
  const int b_bytes = ((b_rows * 128 + 1023) / 1024) * 1024;
  const int b_load_bytes = Dl > 256 ? 512 * 128 : (p.Dloc > 256 ? 256 : p.Dloc) * 128;  // what the TMA boxes deliver
  const int stage_bytes = a_bytes + b_bytes;
  WBars* bar = reinterpret_cast<WBars*>(smem + p.stages * stage_bytes);
  float* zw = reinterpret_cast<float*>(bar + 1);  // [4 warps][D_loc] partial row sums
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int batch = blockIdx.x, mblk = blockIdx.y, k_base = mblk * p.m_tok;
  const int b = batch / p.P, tile = batch - b * p.P;
  const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
  const int rows_per_box = p.m_tok / p.tw;
  const int nk = (p.d + kKC - 1) / kKC;
  const uint32_t ncols = n_mma > 256 ? 512u : n_mma > 128 ? 256u : n_mma > 64 ? 128u : n_mma > 32 ? 64u : 32u;
  const int box_bytes_a = p.m_tok * 128;
  const int box_d0 = Dl > 256 ? 256 : Dl, box_d1 = Dl - box_d0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_d);
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
        const int s = k % p.stages;
        if (k >= p.stages && !mbar_wait(&bar->empty[s], ((k / p.stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sa = smem + s * stage_bytes;
        mbar_expect_tx(&bar->full[s], box_bytes_a + b_load_bytes);
        tma_load_4d(sa, &tm_x, &bar->full[s], k * kKC, tx * p.tw, ty * p.th + mblk * rows_per_box, b);
        tma_load_3d(sa + a_bytes, &tm_d, &bar->full[s], k * kKC, d_base, batch);
        if (box_d1 > 0) tma_load_3d(sa + a_bytes + 256 * 128, &tm_d, &bar->full[s], k * kKC, d_base + 256, batch);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc0 = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, n0);
      const uint32_t idesc1 = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, n1 > 0 ? n1 : 16);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (!mbar_wait(&bar->full[s], (k / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t aa = smem_u32(smem + s * stage_bytes), ba = aa + a_bytes;
#pragma unroll
        for (int kk = 0; kk < kKC / 16; ++kk) {
          const uint64_t ad = smem_desc_sw128(aa + kk * 32, 16, 1024);
          mma_ss(tmem, ad, smem_desc_sw128(ba + kk * 32, 16, 1024), idesc0, k > 0 || kk > 0);
          if (n1 > 0) mma_ss(tmem + 256, ad, smem_desc_sw128(ba + 256 * 128 + kk * 32, 16, 1024), idesc1, k > 0 || kk > 0);
        }
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int quarter = warp & 3;
    const int k_loc = quarter * 32 + lane;              // source row inside this CTA
    const bool valid = k_loc < p.m_tok;
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    float* zrow = zw + quarter * Dl;
    if (mbar_wait(&bar->done, 0, dev_status, abort_flag)) {
      tc_fence_after();
      if (p.raw) {  // scaled logits only: the row's other destination blocks are in other CTAs
        float* dst = shares + ((size_t)batch * p.Nloc + k_base + (valid ? k_loc : 0)) * p.Dloc + d_base;
        for (int i0 = 0; i0 < Dl; i0 += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + i0, r);
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              if (i0 + e < Dl)
                *reinterpret_cast<float4*>(dst + i0 + e) =
                    make_float4(__uint_as_float(r[e]) * p.scale_log2, __uint_as_float(r[e + 1]) * p.scale_log2,
                                __uint_as_float(r[e + 2]) * p.scale_log2, __uint_as_float(r[e + 3]) * p.scale_log2);
          }
        }
      } else {
      // pass 1: maximum logit over the destinations
      float mx = -INFINITY;
      for (int i0 = 0; i0 < p.Dloc; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (i0 + e < p.Dloc) mx = fmaxf(mx, __uint_as_float(r[e]));
      }
      const float neg_m = -mx * p.scale_log2;
      // pass 2: denominator
      float sum = 0.f;
      for (int i0 = 0; i0 < p.Dloc; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (i0 + e < p.Dloc) sum += fast_exp2(fmaf(__uint_as_float(r[e]), p.scale_log2, neg_m));
      }
      const float inv = valid ? 1.f / sum : 0.f;
      // pass 3: shares, their store, and the per-warp column sums
      float* dst = shares + ((size_t)batch * p.Nloc + k_base + (valid ? k_loc : 0)) * p.Dloc;
      for (int i0 = 0; i0 < p.Dloc; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
        float a[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float v = fast_exp2(fmaf(__uint_as_float(r[e]), p.scale_log2, neg_m)) * inv;
          a[e] = (valid && i0 + e < p.Dloc) ? v : 0.f;
        }
        if (valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            if (i0 + e < p.Dloc) *reinterpret_cast<float4*>(dst + i0 + e) = make_float4(a[e], a[e + 1], a[e + 2], a[e + 3]);
        }
        // transpose-reduce: afterwards lane c holds the sum over the warp's 32 rows of column i0 + c
#pragma unroll
        for (int off = 16, n = 32; off >= 1; off >>= 1, n >>= 1) {
          const bool upper = (lane & off) != 0;
#pragma unroll
          for (int c = 0; c < n / 2; ++c) {
            const float send = upper ? a[c] : a[c + n / 2];
            const float keep = upper ? a[c + n / 2] : a[c];
            a[c] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
        if (i0 + lane < p.Dloc) zrow[i0 + lane] = a[0];
      }
      }  // !raw
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps
    const int t = threadIdx.x - 64;
    float* zout = zpart + ((size_t)batch * gridDim.y + mblk) * p.Dloc;
    if (!p.raw)
      for (int i = t; i < p.Dloc; i += 128) zout[i] = (zw[i] + zw[p.Dloc + i]) + (zw[2 * p.Dloc + i] + zw[3 * p.Dloc + i]);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

// ------------------------------------------------------------------------------------------------
// The whole of Sec. 4.2.1 for one tile in one CTA (tiles of at most 256 tokens and 256
// destinations): logits on the tensor cores for both 128-source blocks of the tile (one
// accumulator each), softmax over the destinations in registers, the destinations' row sums added
// up across the tile through shared memory, and the row normalisation 1/Z_i applied as the
// accumulators are read a last time: A~^T leaves the kernel as its hi and lo bf16 planes, and the
// fp32 shares never exist in memory.
//   kMB: 128-source blocks per tile (1 or 2).  Warp 0 TMA, warp 1 MMA, then four epilogue warps
//   per source block (thread = source token = tensor-memory lane).
//   kPair (with kMB = 1): a tile of two source blocks is shared by the two CTAs of a cluster, one block each,
//   which send each other their halves of the row sums (a store into the peer's shared memory per
//   destination, counted on a barrier of the peer's) - for launches of few tiles, where one CTA per tile would
//   leave most SMs idle and each CTA bound by what one SM takes in.
// ------------------------------------------------------------------------------------------------
template <int kMB, bool kPair = false>
__global__ void __launch_bounds__(64 + 128 * kMB, 1)
weights_fused_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_d,
                     __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wu, const WParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int Dl = p.Dloc;
  const int n_mma = (Dl + 15) & ~15;  // MMA N: destinations padded to 16
  const int a_bytes = 128 * 128;      // one source block of a stage (only m_tok rows are loaded)
  const int b_bytes = ((((Dl + 7) & ~7) * 128 + 1023) / 1024) * 1024;
  const int stage_bytes = kMB * a_bytes + b_bytes;
  WBars* bar = reinterpret_cast<WBars*>(smem + p.stages * stage_bytes);
  float* zw = reinterpret_cast<float*>(bar + 1);  // [4 kMB warps][D_loc] partial row sums
  float* zinv = zw + 4 * kMB * Dl;                // [D_loc] reciprocal row sums of the tile
  float* zpeer = zinv + Dl;                       // [D_loc] paired form: the peer block's row sums
  static_assert(!kPair || kMB == 1, "the paired form has one source block per CTA");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int batch = kPair ? blockIdx.x >> 1 : blockIdx.x;
  const int half = kPair ? (int)(blockIdx.x & 1) : 0;  // = rank in the cluster: the tile's source block of this CTA
  const int b = batch / p.P, tile = batch - b * p.P;
  const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
  const int rows_per_box = p.m_tok / p.tw;
  const int nk = (p.d + kKC - 1) / kKC;
  const uint32_t ncols_mb = n_mma > 128 ? 256u : n_mma > 64 ? 128u : n_mma > 32 ? 64u : 32u;
  const uint32_t ncols = kMB * ncols_mb;  // a power of two again (kMB is 1 or 2)

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    mbar_init(&bar->z_in, 128);  // every epilogue thread of the peer arrives once
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_d);
  }
  dependency_wait();  // before tensor memory is held and before any global access
  if (threadIdx.x == 0) release_dependents();
  if (warp == 1) tmem_alloc(&bar->tmem_base, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (kPair) cluster_sync();  // the peer's barrier is initialised before anything is sent to it
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 0) {
    if (elect_one()) {
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (k >= p.stages && !mbar_wait(&bar->empty[s], ((k / p.stages) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sa = smem + s * stage_bytes;
        mbar_expect_tx(&bar->full[s], kMB * p.m_tok * 128 + Dl * 128);
        for (int mb = 0; mb < kMB; ++mb)
          tma_load_4d(sa + mb * a_bytes, &tm_x, &bar->full[s], k * kKC, tx * p.tw, ty * p.th + (mb + half) * rows_per_box, b);
        tma_load_3d(sa + kMB * a_bytes, &tm_d, &bar->full[s], k * kKC, 0, batch);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, n_mma);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % p.stages;
        if (!mbar_wait(&bar->full[s], (k / p.stages) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t aa = smem_u32(smem + s * stage_bytes), ba = aa + kMB * a_bytes;
#pragma unroll
        for (int mb = 0; mb < kMB; ++mb)
#pragma unroll
          for (int kk = 0; kk < kKC / 16; ++kk)
            mma_ss(tmem + mb * ncols_mb, smem_desc_sw128(aa + mb * a_bytes + kk * 32, 16, 1024),
                   smem_desc_sw128(ba + kk * 32, 16, 1024), idesc, k > 0 || kk > 0);
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    const int mb = (warp - 2) >> 2, quarter = warp & 3;
    const int k_loc = quarter * 32 + lane;  // source row inside its block = tensor-memory lane
    const bool valid = k_loc < p.m_tok;
    const uint32_t taddr = tmem + mb * ncols_mb + ((uint32_t)(quarter * 32) << 16);
    float* zrow = zw + (mb * 4 + quarter) * Dl;
    float neg_m = 0.f, inv = 0.f;
    const bool ok = mbar_wait(&bar->done, 0, dev_status, abort_flag);
    if (ok) {
      tc_fence_after();
      // pass 1: maximum logit over the destinations
      float mx = -INFINITY;
      for (int i0 = 0; i0 < Dl; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (i0 + e < Dl) mx = fmaxf(mx, __uint_as_float(r[e]));
      }
      neg_m = -mx * p.scale_log2;
      // pass 2: denominator of the token's softmax
      float sum = 0.f;
      for (int i0 = 0; i0 < Dl; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (i0 + e < Dl) sum += fast_exp2(fmaf(__uint_as_float(r[e]), p.scale_log2, neg_m));
      }
      inv = valid ? 1.f / sum : 0.f;
      // pass 3: the shares' sums over this warp's 32 source tokens, per destination
      for (int i0 = 0; i0 < Dl; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
        float a[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float v = fast_exp2(fmaf(__uint_as_float(r[e]), p.scale_log2, neg_m)) * inv;
          a[e] = (valid && i0 + e < Dl) ? v : 0.f;
        }
        // transpose-reduce: afterwards lane c holds the sum over the warp's 32 rows of column i0 + c
#pragma unroll
        for (int off = 16, n = 32; off >= 1; off >>= 1, n >>= 1) {
          const bool upper = (lane & off) != 0;
#pragma unroll
          for (int c = 0; c < n / 2; ++c) {
            const float send = upper ? a[c] : a[c + n / 2];
            const float keep = upper ? a[c + n / 2] : a[c];
            a[c] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
        if (i0 + lane < Dl) zrow[i0 + lane] = a[0];
      }
    }
    // the tile's row sums: warps of a block pairwise, then the blocks in order (a fixed order: the
    // result does not depend on scheduling); a row sum that underflowed to 0 gives a zero row
    asm volatile("bar.sync 1, %0;" ::"n"(128 * kMB) : "memory");
    if (kPair) {
      // this block's sums go to the peer, the peer's arrive here; both add block 0 + block 1 in that order
      const uint32_t peer = (uint32_t)(half ^ 1);
      const uint32_t peer_z = peer_addr(smem_u32(zpeer), peer);
      for (int i = threadIdx.x - 64; i < Dl; i += 128) {
        const float* q = zw + i;
        const float z = (q[0] + q[Dl]) + (q[2 * Dl] + q[3 * Dl]);
        zinv[i] = z;  // own half, for now
        st_peer_f32(peer_z + 4u * (uint32_t)i, z);
      }
      mbar_arrive_peer(peer_addr(smem_u32(&bar->z_in), peer));
      const bool got = mbar_wait_cluster(&bar->z_in, 0, dev_status, abort_flag);
      for (int i = threadIdx.x - 64; i < Dl; i += 128) {
        const float z = !got ? 0.f : half == 0 ? zinv[i] + zpeer[i] : zpeer[i] + zinv[i];
        zinv[i] = z > 0.f ? 1.f / z : 0.f;
      }
    } else {
      for (int i = threadIdx.x - 64; i < Dl; i += 128 * kMB) {
        float z = 0.f;
#pragma unroll
        for (int m = 0; m < kMB; ++m) {
          const float* q = zw + m * 4 * Dl + i;
          z += (q[0] + q[Dl]) + (q[2 * Dl] + q[3 * Dl]);
        }
        zinv[i] = z > 0.f ? 1.f / z : 0.f;
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(128 * kMB) : "memory");
    if (ok && valid) {
      // pass 4: A~_ik = A_ik / Z_i, written as row k of A~^T [N_loc][D_loc], hi plane then lo plane
      const size_t plane = (size_t)p.Nloc * Dl;
      const size_t row = (size_t)((mb + half) * p.m_tok + k_loc) * Dl;
      __nv_bfloat16* t_hi = w + (size_t)batch * 2 * plane + row;
      __nv_bfloat16* u_hi = wu ? wu + (size_t)batch * 2 * plane + row : nullptr;
      for (int i0 = 0; i0 < Dl; i0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + i0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e0 = 0; e0 < 32; e0 += 8) {
          if (i0 + e0 >= Dl) break;  // D_loc is a multiple of 8
          __align__(16) __nv_bfloat16 hi[8], lo[8], uh[8], ul[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float a = fast_exp2(fmaf(__uint_as_float(r[e0 + e]), p.scale_log2, neg_m)) * inv;
            const float v = a * zinv[i0 + e0 + e];
            hi[e] = __float2bfloat16_rn(v);
            lo[e] = __float2bfloat16_rn(v - __bfloat162float(hi[e]));
            uh[e] = __float2bfloat16_rn(a);
            ul[e] = __float2bfloat16_rn(a - __bfloat162float(uh[e]));
          }
          *reinterpret_cast<uint4*>(t_hi + i0 + e0) = *reinterpret_cast<const uint4*>(hi);
          *reinterpret_cast<uint4*>(t_hi + plane + i0 + e0) = *reinterpret_cast<const uint4*>(lo);
          if (u_hi) {
            *reinterpret_cast<uint4*>(u_hi + i0 + e0) = *reinterpret_cast<const uint4*>(uh);
            *reinterpret_cast<uint4*>(u_hi + plane + i0 + e0) = *reinterpret_cast<const uint4*>(ul);
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
  if (kPair) cluster_sync();  // neither CTA's shared memory goes away while the other could still write to it
}

__global__ void __launch_bounds__(256)
weights_normalise_kernel(const float* __restrict__ shares, const float* __restrict__ zpart, __nv_bfloat16* __restrict__ w,
                         __nv_bfloat16* __restrict__ wu, int Nloc, int Dloc, int mblocks) {
  // wu (may be null): the shares themselves, A^T, in the same two-plane layout
  // grid (blocks over the tile's [N_loc][D_loc] plane in groups of four destinations, tile)
  extern __shared__ float zs[];  // reciprocal row sums of the tile's D_loc destinations
  dependency_wait();  // launched with programmatic stream serialisation
  if (threadIdx.x == 0) release_dependents();
  const size_t batch = blockIdx.y;
  for (int i = threadIdx.x; i < Dloc; i += blockDim.x) {
    float z = 0.f;
    for (int mb = 0; mb < mblocks; ++mb) z += zpart[(batch * mblocks + mb) * Dloc + i];
    zs[i] = z > 0.f ? 1.f / z : 0.f;  // a row sum that underflowed to 0 gives a zero row
  }
  __syncthreads();
  const int plane = Nloc * Dloc;
  const float4* src = reinterpret_cast<const float4*>(shares + batch * plane);
  __nv_bfloat16* t = w + batch * 2 * plane;
  for (int q = blockIdx.x * blockDim.x + threadIdx.x; q < plane / 4; q += gridDim.x * blockDim.x) {
    const int r = q * 4, i = r % Dloc;  // D_loc is a multiple of 4: the four stay in one row
    const float4 a = src[q];
    const float in[4] = {a.x, a.y, a.z, a.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float v = in[e] * zs[i + e];
      hi[e] = __float2bfloat16_rn(v);
      lo[e] = __float2bfloat16_rn(v - __bfloat162float(hi[e]));
    }
    *reinterpret_cast<uint2*>(t + r) = *reinterpret_cast<const uint2*>(hi);
    *reinterpret_cast<uint2*>(t + plane + r) = *reinterpret_cast<const uint2*>(lo);
    if (wu) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        hi[e] = __float2bfloat16_rn(in[e]);
        lo[e] = __float2bfloat16_rn(in[e] - __bfloat162float(hi[e]));
      }
      __nv_bfloat16* u = wu + batch * 2 * plane;
      *reinterpret_cast<uint2*>(u + r) = *reinterpret_cast<const uint2*>(hi);
      *reinterpret_cast<uint2*>(u + plane + r) = *reinterpret_cast<const uint2*>(lo);
    }
  }
}

// Softmax over the destination axis for rows of scaled logits (log2 domain) that span several
// destination blocks: shares[row][i] <- 2^(v_i - max) / sum.  One warp per source row, 32 rows per
// CTA; the CTA then leaves, per destination, the sum of its 32 rows of shares in zblk (rows added in
// row order, so the result does not depend on scheduling).
constexpr int kSoftmaxRows = 32;
__global__ void __launch_bounds__(256)
softmax_rows_kernel(float* __restrict__ shares, float* __restrict__ zblk, int Nloc, int Dloc) {
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t batch = blockIdx.y;
  const int row0 = blockIdx.x * kSoftmaxRows;
  for (int rr = 0; rr < kSoftmaxRows / 8; ++rr) {
    const int row = row0 + warp * (kSoftmaxRows / 8) + rr;
    if (row >= Nloc) break;
    float4* v = reinterpret_cast<float4*>(shares + (batch * Nloc + row) * Dloc);
    float mx = -INFINITY;
    for (int q = lane; q < Dloc / 4; q += 32) {
      const float4 a = v[q];
      mx = fmaxf(fmaxf(mx, fmaxf(a.x, a.y)), fmaxf(a.z, a.w));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    for (int q = lane; q < Dloc / 4; q += 32) {
      const float4 a = v[q];
      sum += (fast_exp2(a.x - mx) + fast_exp2(a.y - mx)) + (fast_exp2(a.z - mx) + fast_exp2(a.w - mx));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = 1.f / sum;
    for (int q = lane; q < Dloc / 4; q += 32) {
      float4 a = v[q];
      a.x = fast_exp2(a.x - mx) * inv;
      a.y = fast_exp2(a.y - mx) * inv;
      a.z = fast_exp2(a.z - mx) * inv;
      a.w = fast_exp2(a.w - mx) * inv;
      v[q] = a;
    }
  }
  __syncthreads();  // the CTA's rows are final (and visible to the whole CTA)
  const int rows = min(kSoftmaxRows, Nloc - row0);
  const float* base = shares + (batch * Nloc + row0) * Dloc;
  float* out = zblk + (batch * gridDim.x + blockIdx.x) * Dloc;
  for (int i = threadIdx.x; i < Dloc; i += blockDim.x) {
    float acc = 0.f;
    for (int r = 0; r < rows; ++r) acc += base[(size_t)r * Dloc + i];
    out[i] = acc;
  }
}

// z[batch][i] = sum over the row blocks of zblk.  A CTA takes 32 destinations; its eight warps each add an eighth
// of the blocks in block order (four loads in flight at a time), and the eight partial sums are added in warp
// order: a fixed association, so the result does not depend on scheduling, and the chain of dependent loads is
// an eighth as long as one thread per destination would make it.
__global__ void __launch_bounds__(256) z_reduce_kernel(const float* __restrict__ zblk, float* __restrict__ z, int nblk, int Dloc) {
  __shared__ float part[8][32];
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 32 + lane;
  const size_t batch = blockIdx.y;
  const int per = (nblk + 7) / 8, b0 = warp * per, b1 = min(nblk, b0 + per);
  float acc = 0.f;
  if (i < Dloc) {
    const float* src = zblk + batch * nblk * Dloc + i;
    int b = b0;
    for (; b + 4 <= b1; b += 4) {
      const float v0 = src[(size_t)b * Dloc], v1 = src[(size_t)(b + 1) * Dloc], v2 = src[(size_t)(b + 2) * Dloc], v3 = src[(size_t)(b + 3) * Dloc];
      acc = (((acc + v0) + v1) + v2) + v3;
    }
    for (; b < b1; ++b) acc += src[(size_t)b * Dloc];
  }
  part[warp][lane] = acc;
  __syncthreads();
  if (warp == 0 && i < Dloc) {
    float t = part[0][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) t += part[w][lane];
    z[batch * Dloc + i] = t;
  }
}

}  // namespace

bool weights_tc_supported(const Geom& g) {
  if (g.f32) return false;
  const int m_tok = g.Nloc < 128 ? g.Nloc : 128;
  if (g.Nloc % m_tok != 0 || m_tok % 8 != 0) return false;
  if (g.tw > m_tok || m_tok % g.tw != 0 || g.th % (m_tok / g.tw) != 0 || g.tw > 256 || m_tok / g.tw > 256) return false;
  if (g.Dloc % 4 != 0) return false;
  if (g.Dloc > 512 && g.Nloc % kSoftmaxRows != 0) return false;  // blocked form: softmax in a second kernel
  return true;
}

size_t weights_tc_scratch_bytes(const Geom& g) {  // gathered destinations + partial row sums
  const size_t tiles = (size_t)g.B * g.P;
  const int m_tok = g.Nloc < 128 ? g.Nloc : 128;
  const size_t dest = tiles * g.Dloc * g.d * 2 + 256;
  if (g.Dloc > 512)  // blocked form: per-row-block sums, then their total
    return dest + tiles * ((size_t)g.Nloc / kSoftmaxRows) * g.Dloc * 4 + 256 + tiles * g.Dloc * 4 + 256;
  return dest + tiles * (g.Nloc / m_tok) * g.Dloc * 4 + 256;
}

cudaError_t launch_weights_tc(const Geom& g, const void* x, const int32_t* idx, void* w, void* wu, float* shares,
                              void* scratch, uint32_t* dev_status, cudaStream_t s) {
  const size_t tiles = (size_t)g.B * g.P;
  WParams p;
  p.P = g.P; p.tiles_x = g.tiles_x; p.th = g.th; p.tw = g.tw; p.W = g.W; p.Nloc = g.Nloc; p.Dloc = g.Dloc; p.d = g.d;
  p.n_all = (int)g.tokens_all();
  p.m_tok = g.Nloc < 128 ? g.Nloc : 128;
  p.scale_log2 = g.logit_scale * 1.4426950408889634f;
  const bool blocked = g.Dloc > 512;  // more destinations than one CTA's tensor memory holds
  p.d_block = blocked ? 512 : g.Dloc;
  p.raw = blocked ? 1 : 0;
  const int mblocks = g.Nloc / p.m_tok;
  __nv_bfloat16* dg = (__nv_bfloat16*)scratch;
  float* zpart = (float*)((char*)scratch + ((tiles * g.Dloc * g.d * 2 + 255) / 256) * 256);

  const int rows_total = (int)(tiles * g.Dloc);
  const long long vecs = (long long)rows_total * (g.d / 8);
  cudaError_t le = launch_dependent(gather_dest_kernel, dim3((unsigned)((vecs + 255) / 256)), dim3(256), 0, s,
                                    (const __nv_bfloat16*)x, idx, dg, p, rows_total);
  count_launch();
  if (le != cudaSuccess) return le;

  CUtensorMap tx, td;
  // One CTA per tile, no fp32 shares in memory.  With two source blocks per tile the fused form halves the
  // CTA count, and a CTA takes in its operands at a few tens of bytes per clock whatever else it does: it
  // wins once there are enough tiles to occupy the SMs anyway (measured: 77 against 91 us on 256 tiles, 30
  // against 26 us on 32 tiles); with one source block per tile it only saves the second kernel.
  const bool fused = g.Dloc <= 256 && g.Dloc % 8 == 0 && (mblocks == 1 || (mblocks == 2 && (int)tiles >= sm_count() / 2));
  // few tiles of two source blocks: the fused form with the tile shared by a cluster of two CTAs (one block each)
  const bool paired = !fused && g.Dloc <= 256 && g.Dloc % 8 == 0 && mblocks == 2;
  const uint64_t xdims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t xstr[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t xbox[4] = {64, (uint32_t)g.tw, (uint32_t)(p.m_tok / g.tw), 1};
  const uint64_t ddims[3] = {(uint64_t)g.d, (uint64_t)g.Dloc, (uint64_t)tiles};
  const uint64_t dstr[2] = {(uint64_t)g.d * 2, (uint64_t)g.Dloc * g.d * 2};
  const uint32_t dbox[3] = {64, (uint32_t)(g.Dloc > 256 ? 256 : g.Dloc), 1};
  if (!encode_tmap_16bit(&tx, x, 4, xdims, xstr, xbox) || !encode_tmap_16bit(&td, dg, 3, ddims, dstr, dbox))
    return cudaErrorInvalidValue;
  const int b_rows = g.Dloc > 256 ? 512 : ((g.Dloc + 7) & ~7);
  const int nk = (g.d + kKC - 1) / kKC;
  if (paired) {
    const int stage_bytes = 128 * 128 + ((b_rows * 128 + 1023) / 1024) * 1024;
    p.stages = (200 * 1024) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages;
    if (p.stages > nk) p.stages = nk;
    const int smem = 1024 + p.stages * stage_bytes + (int)sizeof(WBars) + (4 + 2) * g.Dloc * 4 + 64;
    static std::atomic<unsigned long long> raised_p{0};
    if (cudaError_t e = raise_dynamic_smem(weights_fused_kernel<1, true>, 227 * 1024, raised_p); e != cudaSuccess) return e;
    le = launch_dependent_cluster(weights_fused_kernel<1, true>, dim3((unsigned)(2 * tiles)), dim3(192), (size_t)smem, 2, s, tx, td,
                                  (__nv_bfloat16*)w, (__nv_bfloat16*)wu, p, dev_status);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
  }
  if (fused) {
    const int stage_bytes = mblocks * 128 * 128 + ((b_rows * 128 + 1023) / 1024) * 1024;
    p.stages = (200 * 1024) / stage_bytes;
    p.stages = p.stages > 4 ? 4 : p.stages;
    if (p.stages > nk) p.stages = nk;
    const int smem = 1024 + p.stages * stage_bytes + (int)sizeof(WBars) + (4 * mblocks + 2) * g.Dloc * 4 + 64;
    if (mblocks == 2) {
      static std::atomic<unsigned long long> raised2{0};
      if (cudaError_t e = raise_dynamic_smem(weights_fused_kernel<2>, 227 * 1024, raised2); e != cudaSuccess) return e;
      le = launch_dependent(weights_fused_kernel<2>, dim3((unsigned)tiles), dim3(320), (size_t)smem, s, tx, td,
                            (__nv_bfloat16*)w, (__nv_bfloat16*)wu, p, dev_status);
    } else {
      static std::atomic<unsigned long long> raised1{0};
      if (cudaError_t e = raise_dynamic_smem(weights_fused_kernel<1>, 227 * 1024, raised1); e != cudaSuccess) return e;
      le = launch_dependent(weights_fused_kernel<1>, dim3((unsigned)tiles), dim3(192), (size_t)smem, s, tx, td,
                            (__nv_bfloat16*)w, (__nv_bfloat16*)wu, p, dev_status);
    }
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
  }
  const int stage_bytes = 128 * 128 + ((b_rows * 128 + 1023) / 1024) * 1024;
  p.stages = stage_bytes <= 48 * 1024 ? 4 : 2;
  if (p.stages > nk) p.stages = nk;
  const int smem = 1024 + p.stages * stage_bytes + (int)sizeof(WBars) + 4 * p.d_block * 4 + 64;
  static std::atomic<unsigned long long> smem_raised{0};
  if (cudaError_t e = raise_dynamic_smem(weights_logits_kernel, 200 * 1024, smem_raised); e != cudaSuccess) return e;
  dim3 grid((unsigned)tiles, mblocks, (g.Dloc + p.d_block - 1) / p.d_block);
  le = launch_dependent(weights_logits_kernel, grid, dim3(192), (size_t)smem, s, tx, td, shares, zpart, p, dev_status);
  count_launch();
  if (le != cudaSuccess) return le;
  const float* zsrc = zpart;
  int zblocks = mblocks;
  if (blocked) {  // softmax over the full rows, then the destinations' row sums in two deterministic steps
    const int nrb = g.Nloc / kSoftmaxRows;
    float* zblk = zpart;
    float* z = (float*)((char*)zblk + ((tiles * nrb * g.Dloc * 4 + 255) / 256) * 256);
    le = launch_dependent(softmax_rows_kernel, dim3((unsigned)nrb, (unsigned)tiles), dim3(256), 0, s, shares,
                          zblk, g.Nloc, g.Dloc);
    count_launch();
    if (le != cudaSuccess) return le;
    le = launch_dependent(z_reduce_kernel, dim3((unsigned)((g.Dloc + 31) / 32), (unsigned)tiles), dim3(256), 0, s,
                          (const float*)zblk, z, nrb, g.Dloc);
    count_launch();
    if (le != cudaSuccess) return le;
    zsrc = z;
    zblocks = 1;
  }
  const int quads = g.Nloc * g.Dloc / 4;
  int nblocks = (quads + 1023) / 1024;  // four quads per thread
  nblocks = nblocks < 1 ? 1 : nblocks > 1024 ? 1024 : nblocks;
  static std::atomic<unsigned long long> smem_raised3{0};
  if (g.Dloc * 4 > 48 * 1024) {
    if (cudaError_t e = raise_dynamic_smem(weights_normalise_kernel, 200 * 1024, smem_raised3); e != cudaSuccess) return e;
  }
  le = launch_dependent(weights_normalise_kernel, dim3((unsigned)nblocks, (unsigned)tiles), dim3(256), (size_t)g.Dloc * 4, s,
                        (const float*)shares, zsrc, (__nv_bfloat16*)w, (__nv_bfloat16*)wu, g.Nloc, g.Dloc, zblocks);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace toma
