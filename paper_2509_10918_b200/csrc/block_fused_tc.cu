// One kernel for a whole reuse step of the small-tile block (Algorithm 3 with cached destinations and
// weights): merge, attention over the merged tokens and unmerge without a pass through global memory
// between them.  For tiles of 64 tokens with 32 destinations, 64-wide heads and at most 512 merged
// tokens per image (the 32x32-token SDXL block with 8x8 tiles), where the three separate kernels
// are a few microseconds of work behind three launches.
//
// Merge is linear per channel and local to a tile, and a head's attention needs the merged tokens of
// all tiles but only the head's 64 channels.  So one CTA = (batch, head, 256 merged queries = 8 tiles):
//   A  merges the head's 64 channels of its own 8 tiles into its 256 rows of a [D][64] bf16 matrix in
//      shared memory - K and V of the head.  With 512 merged tokens the head's two CTAs form a cluster,
//      and each sends its rows to the other's copy of the matrix (bulk copies between the shared memories);
//   B  runs the attention of its 256 merged queries (two 128-row query tiles, rows of the same matrix)
//      over the D keys exactly as attention_tc.cu does (S double-buffered in tensor memory, P written
//      over S, [V | 1] operand for the row sums, lazy rescale), except that nothing is loaded: K and V
//      are resident;
//   C  unmerges its 8 tiles' 512 tokens x 64 channels from the normalised accumulators (written to
//      shared memory as bf16, the B operand of the unmerge) and stores them in spatial order (rows staged
//      where K and V were, one TMA store per warp's half tile).
// Both contractions with the weights run on the tensor cores with 128 rows on M by pairing tiles: the
// operand of a pair is block diagonal, a [128 tokens][64 destinations] slab whose row k holds token k's
// 32 weights in the half that belongs to its tile and zeros in the other.  Read MN-major it is the A
// operand of the merge (X_m = A~ X: M = destination, K = token), read K-major it is the A operand of
// the unmerge (Y = A~^T X': M = token, K = destination).  The slab (hi and lo bf16 planes) is built
// from the stored A~^T with ordinary loads and swizzled stores by the softmax warps, which have
// nothing else to do at that time.  A merge MMA has M = 128 = two such 64-destination slabs; the
// pair that belongs to the other half of the accumulator's rows reads a block of zeros instead.
//
// Warps 0..3 / 4..7: softmax of query tile 0 / 1; in A warps 0..3 build slabs and warps 4..7 move
// merged rows from tensor memory to shared memory; in C each group builds and stores its own pairs.
// Warp 8: TMA producer of the token tiles (A only; the four pairs have a stage each).  Warp 9: one elected thread issues every MMA.
#include "attention_core.cuh"
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;
using namespace attn;

namespace {

constexpr int kThreads = 384;
constexpr int kTileTok = 64, kTileDest = 32;  // the tile shape this kernel is written for
constexpr int kPairBytes = 128 * 128;         // one plane of a pair's slab, and one pair of token tiles
constexpr int kZeroBytes = 2048;              // 16 rows x 128 B of zeros: the other half of a merge MMA's A operand
constexpr int kOnesBytes = kBN * 128;
constexpr int kMaxD = 512;                    // merged tokens per image the shared-memory matrix holds

struct FBars {
  uint64_t x_full[4];                    // token tiles of a pair landed (TMA)
  uint64_t slab_full[2], slab_empty[2];  // slab of a pair built (4 warps) / its MMAs are done with it
  uint64_t slab2_full;                   // the extra slab of the unmerge's third pair
  uint64_t acc_full[2];    // merge: a group of four tiles accumulated
  uint64_t kv_ready;       // the merged matrix is complete in shared memory (both CTAs' rows)
  uint64_t kv_sent;        // the peer has received this CTA's rows (they may be overwritten)
  uint64_t s_full[2][2], p_full[2][2];
  uint64_t pv_done[4];     // per key tile: its PV products (both query tiles) have landed
  uint64_t o_done[2];
  uint64_t os_full[2];     // normalised accumulator of a query tile written to shared memory
  uint64_t c_full[2][2];   // unmerge: accumulator of pair (query tile, pair) complete
  uint32_t tmem_base;
  int abort_flag;
};

struct FParams {
  int tiles_x, th, tw, heads, D, units;  // units = D / 256 per (batch, head)
  const __nv_bfloat16* w;  // A~^T planes: [tile][hi, lo][64 tokens][32 destinations]
  float scale_log2;
};

// A thread's row of a pair's slab: the 32 weights (hi and lo plane) of one token of tile ta or ta + 1.
struct SlabRow {
  uint4 v[2][4];
};
__device__ __forceinline__ SlabRow load_slab_row(const FParams& p, int b, int ta, int r /*0..127*/) {
  const int tile = r < kTileTok ? ta : ta + 1, k = r & (kTileTok - 1);
  const size_t row = ((size_t)(2 * (b * (p.D / kTileDest) + tile)) * kTileTok + k) * kTileDest;
  SlabRow w;
#pragma unroll
  for (int pl = 0; pl < 2; ++pl) {
    const uint4* src = reinterpret_cast<const uint4*>(p.w + row + (size_t)pl * kTileTok * kTileDest);
#pragma unroll
    for (int c = 0; c < 4; ++c) w.v[pl][c] = __ldg(src + c);
  }
  return w;
}
// Writes it into `slab` (hi plane, then lo plane kPairBytes further): data in the half of the row that belongs to the
// token's tile, zeros in the other.
__device__ __forceinline__ void store_slab_row(uint8_t* slab, const SlabRow& w, int r) {
  const int side = r >> 6;
#pragma unroll
  for (int pl = 0; pl < 2; ++pl) {
    uint8_t* dst = slab + pl * kPairBytes;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      *reinterpret_cast<uint4*>(dst + sw128_offset(r, side * 4 + c)) = w.v[pl][c];
      *reinterpret_cast<uint4*>(dst + sw128_offset(r, (side ^ 1) * 4 + c)) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

// 64 fp32 of a tensor-memory row -> one 128-byte bf16 row of a swizzled shared-memory tile, scaled.
__device__ __forceinline__ void row_to_smem(uint32_t taddr, uint8_t* tile, int row, float scale) {
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    uint32_t r[32];
    tmem_ld32(taddr + c * 32, r);
    tmem_wait_ld();
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
      uint4 v;
      v.x = pack_bf16_rn(__uint_as_float(r[e]) * scale, __uint_as_float(r[e + 1]) * scale);
      v.y = pack_bf16_rn(__uint_as_float(r[e + 2]) * scale, __uint_as_float(r[e + 3]) * scale);
      v.z = pack_bf16_rn(__uint_as_float(r[e + 4]) * scale, __uint_as_float(r[e + 5]) * scale);
      v.w = pack_bf16_rn(__uint_as_float(r[e + 6]) * scale, __uint_as_float(r[e + 7]) * scale);
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, c * 4 + (e >> 3))) = v;
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
block_fused_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_out, const FParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sKV = smem;                           // [D][128 B]: merged tokens of the head, K-major rows
  uint8_t* sX = sKV + kMaxD * 128;               // 4 x one pair of token tiles; later the two normalised accumulators and a slab
  uint8_t* sZlo = sX + 4 * kPairBytes;           // zeros below the slabs
  uint8_t* sA = sZlo + kZeroBytes;               // 2 x (hi plane, lo plane) of a pair's slab
  uint8_t* sZhi = sA + 4 * kPairBytes;           // zeros above the slabs
  uint8_t* sOnes = sZhi + kZeroBytes;
  FBars* bar = reinterpret_cast<FBars*>(sOnes + kOnesBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.x % p.units, bh = blockIdx.x / p.units, h = bh % p.heads, b = bh / p.heads;
  constexpr int n_pairs = 4;            // pairs of tiles this CTA merges (its unit's 8 tiles) and unmerges
  const int nblk = p.D / kBN;           // key tiles
  const int tiles_x = p.tiles_x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) {
      mbar_init(&bar->x_full[s], 1);
    }
    mbar_init(&bar->slab2_full, 4);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->slab_full[s], 4);
      mbar_init(&bar->slab_empty[s], 1);
      mbar_init(&bar->acc_full[s], 1);
      mbar_init(&bar->o_done[s], 1);
      mbar_init(&bar->os_full[s], 4);
      for (int t = 0; t < 2; ++t) {
        mbar_init(&bar->s_full[s][t], 1);
        mbar_init(&bar->p_full[s][t], 4);
        mbar_init(&bar->c_full[s][t], 1);
      }
    }
    for (int s = 0; s < 4; ++s) mbar_init(&bar->pv_done[s], 1);
    mbar_init(&bar->kv_ready, p.units == 2 ? 5 : 4);  // own warps; the peer's rows arrive as bytes
    bar->abort_flag = 0;
    mbar_fence_init();
    mbar_init(&bar->kv_sent, 1);
    if (p.units == 2) mbar_expect_tx(&bar->kv_ready, 2 * kPairBytes);
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_out);
  }
  for (int e = threadIdx.x; e < kOnesBytes / 4; e += blockDim.x) reinterpret_cast<uint32_t*>(sOnes)[e] = 0x3F803F80u;
  for (int e = threadIdx.x; e < kZeroBytes / 4; e += blockDim.x) {
    reinterpret_cast<uint32_t*>(sZlo)[e] = 0u;
    reinterpret_cast<uint32_t*>(sZhi)[e] = 0u;
  }
  fence_proxy_async();
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  if (warp == 9) tmem_alloc(&bar->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (p.units == 2) cluster_sync();  // the peer's barriers are initialised before anything is sent to it
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;
  // tensor memory: columns 0..255 the four S buffers (the merge accumulators before, the unmerge accumulators
  // after, in the same columns); the attention accumulators (and row sums) from column 256
  constexpr int kColO = 256, kOStride = 96;

  if (warp == 8) {
    // ------------------------------------------------------------------ A: token tiles of every pair
    if (elect_one()) {
      for (int i = 0; i < n_pairs; ++i) {
        const int s = i;
        mbar_expect_tx(&bar->x_full[s], kPairBytes);
        for (int t = 0; t < 2; ++t) {
          const int tile = unit * 8 + 2 * i + t, ty = tile / tiles_x, tx = tile - ty * tiles_x;
          tma_load_4d(sX + s * kPairBytes + t * (kPairBytes / 2), &tm_x, &bar->x_full[s], h * 64, tx * p.tw, ty * p.th, b);
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ every MMA, in program order
    if (elect_one()) {
      bool ok = true;
      // ---- A: X_m rows of four tiles = (pair 0 | zeros) and (zeros | pair 1) times the tokens of the pairs
      constexpr uint32_t idesc_m = idesc_f16(kFmtBF16, kFmtBF16, true, true, 128, 64);
      for (int i = 0; ok && i < n_pairs; ++i) {
        const int s = i & 1, xs = i, g = i >> 1;  // slab stage; token stage; group of four tiles
        if (!mbar_wait(&bar->x_full[xs], 0, dev_status, abort_flag) ||
            !mbar_wait(&bar->slab_full[s], (i >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t xa = smem_u32(sX + xs * kPairBytes);
        const uint32_t t_acc = tmem + g * 64;
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
          const uint32_t sa = smem_u32(sA + (2 * s + pl) * kPairBytes);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {  // 16 tokens per MMA
            // rows 0..63 of the accumulator belong to the group's first pair, rows 64..127 to its second
            const uint32_t slab = sa + kk * 2048;
            const uint64_t ad = (i & 1) == 0 ? smem_desc_sw128(slab, smem_u32(sZhi) - slab, 1024)
                                             : smem_desc_sw128(smem_u32(sZlo), slab - smem_u32(sZlo), 1024);
            mma_ss(t_acc, ad, smem_desc_sw128(xa + kk * 2048, 16, 1024), idesc_m, (i & 1) != 0 || pl > 0 || kk > 0);
          }
        }
        mma_commit(&bar->slab_empty[s]);
        if (i & 1) mma_commit(&bar->acc_full[g]);
      }
      // ---- B: attention of the unit's two query tiles over all D keys of the resident matrix
      if (ok) ok = mbar_wait_cluster(&bar->kv_ready, 0, dev_status, abort_flag);
      if (ok) {
        if (p.units == 2) mbar_arrive_peer(peer_addr(smem_u32(&bar->kv_sent), (uint32_t)(unit ^ 1)));
        tc_fence_after();
        constexpr uint32_t idesc_s = idesc_f16(kFmtBF16, kFmtBF16, false, false, kBM, kBN);
        constexpr uint32_t idesc_o = idesc_f16(kFmtBF16, kFmtBF16, false, true, kBM, 64 + 16);
        const uint32_t kv = smem_u32(sKV);
        const uint64_t kv_desc = smem_desc_sw128(kv, 16, 1024);
        auto issue_s = [&](int n, int q) {
          const uint64_t qd = kv_desc + (uint64_t)(((unit * 256 + q * kBM) * 128) >> 4);
          const uint64_t kd = kv_desc + (uint64_t)((n * kBN * 128) >> 4);
          const uint32_t t_s = tmem + (2 * q + (n & 1)) * kBN;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) mma_ss(t_s, qd + (uint64_t)((kk * 32) >> 4), kd + (uint64_t)((kk * 32) >> 4), idesc_s, kk > 0);
          mma_commit(&bar->s_full[q][n & 1]);
        };
        for (int n = 0; n < 2 && n < nblk; ++n) {
          issue_s(n, 0);
          issue_s(n, 1);
        }
        for (int n = 0; ok && n < nblk; ++n) {
          const int bb = n & 1;
          const uint32_t va = kv + n * kBN * 128;
          const uint64_t vd = smem_desc_sw128(va, smem_u32(sOnes) - va, 1024);  // [V | ones]
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            if (!mbar_wait(&bar->p_full[q][bb], (n >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_o = tmem + kColO + q * kOStride, t_p = tmem + (2 * q + bb) * kBN;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_ts(t_o, t_p + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o, n > 0 || kk > 0);
            if (n + 1 == nblk) mma_commit(&bar->o_done[q]);
            if (q == 1) mma_commit(&bar->pv_done[n & 3]);
            if (n + 2 < nblk) issue_s(n + 2, q);
          }
        }
      }
      // ---- C: unmerge of the unit's four pairs: Y = (pair's slab, K-major) times the pair's 64 normalised rows
      if (ok) {
        constexpr uint32_t idesc_u = idesc_f16(kFmtBF16, kFmtBF16, false, true, 128, 64);
        for (int c = 0; ok && c < 4; ++c) {
          // slabs: pairs 0 and 1 follow phase A in the two slab stages, pair 2 has the extra buffer (the token
          // stages 2 and 3, free since phase A), pair 3 takes the stage of pair 0 after its MMAs
          const int q = c >> 1, gi = c < 2 ? n_pairs + c : n_pairs + 2, s = gi & 1;
          if ((c & 1) == 0 && !mbar_wait(&bar->os_full[q], 0, dev_status, abort_flag)) { ok = false; break; }
          if (!(c == 2 ? mbar_wait(&bar->slab2_full, 0, dev_status, abort_flag)
                       : mbar_wait(&bar->slab_full[s], (gi >> 1) & 1, dev_status, abort_flag))) { ok = false; break; }
          tc_fence_after();
          const uint32_t os = smem_u32(sX + q * kPairBytes) + (c & 1) * 64 * 128;  // the pair's 64 rows
          const uint32_t t_c = tmem + (2 * q + (c & 1)) * kBN;
          const uint32_t slab0 = c == 2 ? smem_u32(sX + 2 * kPairBytes) : smem_u32(sA + 2 * s * kPairBytes);
#pragma unroll
          for (int pl = 0; pl < 2; ++pl) {
            const uint32_t sa = slab0 + pl * kPairBytes;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)  // 16 destinations per MMA
              mma_ss(t_c, smem_desc_sw128(sa + kk * 32, 16, 1024), smem_desc_sw128(os + kk * 2048, 16, 1024), idesc_u, pl > 0 || kk > 0);
          }
          if (c == 0) mma_commit(&bar->slab_empty[s]);
          mma_commit(&bar->c_full[q][c & 1]);
        }
      }
    }
  } else if (warp < 8) {
    const int q = warp >> 2, quarter = warp & 3, r = quarter * 32 + lane;  // r: row of this thread's 128-row tiles
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    bool ok = true;
    // ------------------------------------------------------------------ A
    if (q == 0) {
      // slabs of all pairs, then (same stages, same barriers) of the first two pairs of the unmerge; a pair's
      // weights are requested before the wait for its stage, so that their latency passes under it
      constexpr int n_build = n_pairs + 2;
      SlabRow w0 = load_slab_row(p, b, unit * 8, r), w1 = load_slab_row(p, b, unit * 8 + 2, r);
#pragma unroll
      for (int i = 0; i < n_build; ++i) {
        const int s = i & 1;
        const SlabRow cur = w0;
        w0 = w1;
        if (i + 2 < n_build) w1 = load_slab_row(p, b, unit * 8 + 2 * ((i + 2) % n_pairs), r);
        if (i >= 2 && !mbar_wait(&bar->slab_empty[s], ((i >> 1) - 1) & 1, dev_status, abort_flag)) { ok = false; break; }
        store_slab_row(sA + 2 * s * kPairBytes, cur, r);
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar->slab_full[s]);
      }
    } else {
      // merged rows of every group of four tiles: tensor memory -> bf16 rows of the shared matrix
      const uint32_t peer = (uint32_t)(unit ^ 1);
      for (int g = 0; g < n_pairs / 2; ++g) {
        if (!mbar_wait(&bar->acc_full[g], 0, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        uint8_t* rows = sKV + (unit * 2 + g) * kPairBytes + quarter * 4096;  // this warp's 32 rows
        row_to_smem(tmem + lane_addr + g * 64, sKV + (unit * 2 + g) * kPairBytes, r, 1.f);
        fence_proxy_async();  // read by the tensor cores and by the copy
        __syncwarp();
        if (p.units == 2 && lane == 0) copy_to_peer(peer_addr(smem_u32(rows), peer), rows, 4096, peer_addr(smem_u32(&bar->kv_ready), peer));
      }
      tc_fence_before();
      if (lane == 0) mbar_arrive(&bar->kv_ready);
      // the unmerge's third pair, into the token stages 2 and 3: every merge MMA has completed (the last group's
      // accumulator was complete), so nothing reads them any more
      if (ok) {
        store_slab_row(sX + 2 * kPairBytes, load_slab_row(p, b, unit * 8 + 4, r), r);
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar->slab2_full);
      }
    }
    // ------------------------------------------------------------------ B
    const uint32_t ob = tmem + lane_addr + kColO + q * kOStride;
    float m_used = -INFINITY, l = 0.f;
    for (int n = 0; ok && n < nblk; ++n) {
      const int bb = n & 1;
      const uint32_t sb = tmem + lane_addr + (2 * q + bb) * kBN;
      if (!mbar_wait(&bar->s_full[q][bb], (n >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
      tc_fence_after();
      ok = softmax_tile<64, true, false>(sb, ob, p.scale_log2, kBN, n, m_used, l, &bar->pv_done[(n + 3) & 3], (uint32_t)(((n - 1) >> 2) & 1),
                                         dev_status, abort_flag);
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->p_full[q][bb]);
    }
    // normalised accumulator -> bf16 rows in shared memory (the unmerge's B operand)
    SlabRow w3;
    if (q == 1) w3 = load_slab_row(p, b, unit * 8 + 6, r);  // the unmerge's fourth pair; needed after the next wait
    if (ok) ok = mbar_wait(&bar->o_done[q], 0, dev_status, abort_flag);
    if (ok) {
      tc_fence_after();
      uint32_t rs[16];
      tmem_ld16(ob + 64, rs);
      tmem_wait_ld();
      row_to_smem(ob, sX + q * kPairBytes, r, 1.f / __uint_as_float(rs[0]));
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->os_full[q]);
    }
    // ------------------------------------------------------------------ C
    if (ok && q == 1) {  // the fourth pair's slab takes the stage of the first once its MMAs are done
      const int gi = n_pairs + 2, s = gi & 1;
      ok = mbar_wait(&bar->slab_empty[s], ((gi >> 1) - 1) & 1, dev_status, abort_flag);
      if (ok) {
        store_slab_row(sA + 2 * s * kPairBytes, w3, r);
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar->slab_full[s]);
      }
    }
    // the rows of K and V become the staging area of the output; the peer must have received its copy of them
    if (ok && p.units == 2) ok = mbar_wait_cluster(&bar->kv_sent, 0, dev_status, abort_flag);
    for (int c = 2 * q; ok && c < 2 * q + 2; ++c) {
      if (!mbar_wait(&bar->c_full[q][c & 1], 0, dev_status, abort_flag)) { ok = false; break; }
      tc_fence_after();
      uint8_t* stage = sKV + c * kPairBytes;  // K and V are no longer read: every MMA before this accumulator's has completed
      row_to_smem(tmem + lane_addr + (2 * q + (c & 1)) * kBN, stage, r, 1.f);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {  // the warp's 32 tokens are the upper or lower half of a tile
        const int tile = unit * 8 + 2 * c + (quarter >> 1), ty = tile / tiles_x, tx = tile - ty * tiles_x;
        tma_store_4d(&tm_out, stage + quarter * 4096, h * 64, tx * p.tw, ty * p.th + (quarter & 1) * (p.th / 2), b);
        tma_store_commit();
      }
    }
    if (lane == 0) tma_store_wait_read();  // shared memory must outlive the engine's reads
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (p.units == 2) cluster_sync();  // neither CTA's shared memory goes away while the other could still write to it
}

constexpr int kFusedSmem = 1024 + kMaxD * 128 + 4 * kPairBytes + 2 * kZeroBytes + 4 * kPairBytes + kOnesBytes + 512;

}  // namespace

// Shapes the fused reuse-step kernel is written for (see the top of this file).
bool block_fused_supported(const Geom& g) {
  if (g.f32 || g.global_merge || g.n_extra != 0 || g.unmerge_mode != TOMA_UNMERGE_TRANSPOSE) return false;
  if (g.dh != 64 || g.Nloc != kTileTok || g.Dloc != kTileDest) return false;
  if (g.tw > 32 || 64 % g.tw != 0 || g.th != 64 / g.tw) return false;  // a tile is one 4-D TMA box of 64 tokens, half a tile a box too
  if (g.D > kMaxD || g.D % 256 != 0 || g.P % 4 != 0) return false;     // whole 256-query units, whole groups of four tiles
  return true;
}

// Whether this device can hold the kernel's launch at all: the shared memory of one CTA and, for 512 merged
// tokens, two such CTAs as a cluster.  Asked once per device (a host-side occupancy query, nothing is launched);
// toma_block takes the three-kernel form where the answer is no.
bool block_fused_launchable(const Geom& g) {
  static std::atomic<unsigned long long> raised{0};
  static std::atomic<int> answer[64][2];  // per device and cluster size - 1: 0 unknown, 1 yes, 2 no
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  const int units = g.D / 256;
  const int known = answer[dev][units - 1].load(std::memory_order_relaxed);
  if (known) return known == 1;
  bool ok = raise_dynamic_smem(block_fused_kernel, kFusedSmem, raised) == cudaSuccess;
  if (ok) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * units);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kFusedSmem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)units;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    ok = cudaOccupancyMaxActiveClusters(&clusters, block_fused_kernel, &cfg) == cudaSuccess && clusters >= 1;
  }
  if (!ok) (void)cudaGetLastError();  // a failed query is an answer, not an error of the caller's stream
  answer[dev][units - 1].store(ok ? 1 : 2, std::memory_order_relaxed);
  return ok;
}

cudaError_t launch_block_fused(const Geom& g, const void* w, const void* x, void* out, uint32_t* dev_status, cudaStream_t s) {
  static_assert(sizeof(FBars) <= 512, "barrier block outgrew its reservation");
  CUtensorMap tx, to;
  const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t strides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t box[4] = {64, (uint32_t)g.tw, (uint32_t)g.th, 1};
  const uint32_t box_out[4] = {64, (uint32_t)g.tw, (uint32_t)g.th / 2, 1};  // a warp stores half a tile
  if (!encode_tmap_16bit(&tx, x, 4, dims, strides, box) || !encode_tmap_16bit(&to, out, 4, dims, strides, box_out)) return cudaErrorInvalidValue;
  FParams p;
  p.tiles_x = g.tiles_x; p.th = g.th; p.tw = g.tw;
  p.heads = g.heads; p.D = g.D; p.units = g.D / 256;
  p.w = (const __nv_bfloat16*)w;
  p.scale_log2 = 1.4426950408889634f / 8.0f;  // log2(e) / sqrt(64)
  static std::atomic<unsigned long long> raised{0};
  cudaError_t e = raise_dynamic_smem(block_fused_kernel, kFusedSmem, raised);
  if (e != cudaSuccess) return e;
  e = launch_dependent_cluster(block_fused_kernel, dim3(g.B * g.heads * p.units), dim3(kThreads), (size_t)kFusedSmem, p.units, s, tx, to, p, dev_status);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace toma
