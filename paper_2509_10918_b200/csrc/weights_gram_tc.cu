// Merge weights out of the raw Gram matrix (Sec. 4.2.1), for the refresh steps of toma_block on few, large
// tiles.  The logit of source token k and destination i is <x_idx_i, x_k> / (tau sqrt(d)): an entry of
// G = X X^T of the tile, whichever tokens the selection picks.  So G does not depend on the selection, and
// while the greedy rounds (Algorithm 2) occupy one SM per tile for their D_loc sequential rounds, the other
// SMs compute it:
//   gram_raw_kernel   G = X X^T per tile on the tensor cores (fp32, [tile][N_loc][N_loc]), launched BEHIND the
//                     greedy kernel with programmatic stream serialisation.  The greedy kernel releases its
//                     dependents as soon as its own inputs are complete, so this kernel's CTAs start on the idle
//                     SMs at once; they read only X (complete long before) and wait for the greedy kernel at
//                     their very END, so that whatever follows in the stream still follows the selection.
//   weights_gram_kernel  a cluster of CTAs per tile, one per 64 source tokens: the D_loc rows G[idx_i] (its strip
//                     of them) into shared memory, softmax over the destinations per source token, the
//                     destinations' row sums exchanged between the CTAs through distributed shared memory,
//                     A~^T as hi and lo planes - no gathered copy of the destinations, no second contraction.
// G lies where the quantised tokens were (they are dead once the fixed-point Gram exists).
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;

namespace {

constexpr int kKC = 64;       // contraction elements per stage
constexpr int kStagesG = 4;
constexpr int kMaxTok = 256;  // tokens per tile both kernels cover

struct GBars {
  uint64_t full[kStagesG], empty[kStagesG], done;
  uint32_t tmem_base;
  int abort_flag;
};

struct GParams {
  int P, tiles_x, th, tw, Nloc, Dloc, d;
  float scale_log2;  // log2(e) / (tau * sqrt(d))
};

__global__ void __launch_bounds__(192, 1)
gram_raw_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, float* __restrict__ G,
                const GParams p, uint32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int Nloc = p.Nloc;
  const int a_bytes = 128 * 128, b_bytes = Nloc * 128, stage_bytes = a_bytes + b_bytes;
  GBars* bar = reinterpret_cast<GBars*>(smem + kStagesG * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_b = blockIdx.x, m0 = blockIdx.y * 128;
  const int b = tile_b / p.P, tile = tile_b - b * p.P;
  const int ty = tile / p.tiles_x, tx = tile - ty * p.tiles_x;
  const int nk = p.d / kKC;
  const uint32_t ncols = Nloc > 128 ? 256u : Nloc > 64 ? 128u : 64u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStagesG; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    mbar_init(&bar->done, 1);
    bar->abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
  }
  // No wait here: the kernel before this one in the stream (the greedy rounds) neither writes anything this
  // kernel reads nor reads what it writes, and it released its dependents only when everything earlier was complete.
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
        const int s = k % kStagesG;
        if (k >= kStagesG && !mbar_wait(&bar->empty[s], ((k / kStagesG) - 1) & 1, dev_status, abort_flag)) break;
        uint8_t* sa = smem + s * stage_bytes;
        mbar_expect_tx(&bar->full[s], stage_bytes);
        tma_load_4d(sa, &tm_a, &bar->full[s], k * kKC, tx * p.tw, ty * p.th + m0 / p.tw, b);
        tma_load_4d(sa + a_bytes, &tm_b, &bar->full[s], k * kKC, tx * p.tw, ty * p.th, b);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(kFmtBF16, kFmtBF16, false, false, 128, Nloc);
      bool ok = true;
      for (int k = 0; k < nk; ++k) {
        const int s = k % kStagesG;
        if (!mbar_wait(&bar->full[s], (k / kStagesG) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t aa = smem_u32(smem + s * stage_bytes), ba = aa + a_bytes;
#pragma unroll
        for (int kk = 0; kk < kKC / 16; ++kk)
          mma_ss(tmem, smem_desc_sw128(aa + kk * 32, 16, 1024), smem_desc_sw128(ba + kk * 32, 16, 1024), idesc, k > 0 || kk > 0);
        mma_commit(&bar->empty[s]);
      }
      if (ok) mma_commit(&bar->done);
    }
  } else {
    // rows leave tensor memory one per thread; they are staged in shared memory (the ring is free by then) with
    // an odd pitch and written out a row at a time by whole warps, so that the stores are whole lines
    const int quarter = warp & 3, r_in = quarter * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    float* stage = reinterpret_cast<float*>(smem);
    const int pitch = Nloc + 1;
    if (__all_sync(0xffffffffu, mbar_wait(&bar->done, 0, dev_status, abort_flag))) {
      tc_fence_after();
      for (int c0 = 0; c0 < Nloc; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(taddr + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) stage[r_in * pitch + c0 + e] = __uint_as_float(v[e]);
      }
      __syncwarp();  // a warp writes out the 32 rows it staged itself
      float* out = G + ((size_t)tile_b * Nloc + m0 + quarter * 32) * Nloc;
      for (int r = 0; r < 32; ++r) {
        if (m0 + quarter * 32 + r >= Nloc) break;
        const float* src = stage + (quarter * 32 + r) * pitch;
        for (int c = lane; c < Nloc; c += 32) out[(size_t)r * Nloc + c] = src[c];
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
  // Only now the kernel before this one in the stream: this grid is complete when the selection is.
  dependency_wait();
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// A cluster of N_loc / 64 CTAs per tile, 256 threads each: CTA r of the cluster owns the source tokens
// 64 r .. 64 r + 63 (a 64-column strip of the rows G[idx_i]); four threads share a column, each with a quarter of
// the destinations.  The destinations' row sums need all sources: every CTA sends its strip's sums to its peers
// (one store into each peer's shared memory per destination, counted on a barrier of the peer's) and adds the
// strips' sums in rank order.
constexpr int kStrip = 64;

struct WgBars {
  uint64_t z_in;  // the peers' row sums have arrived
  int abort_flag;
};

__global__ void __launch_bounds__(256)
weights_gram_kernel(const float* __restrict__ G, const int32_t* __restrict__ idx, __nv_bfloat16* __restrict__ w, const GParams p,
                    uint32_t* dev_status) {
  extern __shared__ float wg_smem[];
  const int Nloc = p.Nloc, Dl = p.Dloc;
  constexpr int pitch = kStrip + 1;
  const int n_cta = Nloc / kStrip;            // CTAs of the cluster = strips of the tile
  float* A = wg_smem;                         // [D_loc][pitch]: logits, then shares, of this strip
  float* zpart = A + Dl * pitch;              // [n_cta][D_loc]: every strip's row sums (slot r filled by CTA r)
  float* zinv = zpart + n_cta * Dl;           // [D_loc]
  float* red = zinv + Dl;                     // [4][kStrip]
  int* sel = reinterpret_cast<int*>(red + 4 * kStrip);  // [D_loc]
  WgBars* bar = reinterpret_cast<WgBars*>(sel + ((Dl + 1) & ~1));
  const int rank = (int)cluster_rank(), tile_b = blockIdx.x / n_cta;
  const int t = threadIdx.x, c = t % kStrip, part = t / kStrip, warp = t >> 5, lane = t & 31;
  if (t == 0) {
    mbar_init(&bar->z_in, (uint32_t)((n_cta - 1) * 128));
    bar->abort_flag = 0;
    mbar_fence_init();
  }
  dependency_wait();  // G and the selection are complete
  if (t == 0) release_dependents();
  for (int i = t; i < Dl; i += blockDim.x) sel[i] = idx[(size_t)tile_b * Dl + i];
  __syncthreads();
  cluster_sync();  // the peers' barriers are initialised before anything is sent to them
  // this strip of the rows G[idx_i]: 64 consecutive threads read 256 consecutive bytes
  const float* Gt = G + (size_t)tile_b * Nloc * Nloc + rank * kStrip + c;
  for (int i0 = part; i0 < Dl; i0 += 128) {  // 32 loads in flight per thread, then their stores
    float v[32];
#pragma unroll
    for (int u = 0; u < 32; ++u) {
      const int i = i0 + 4 * u;
      v[u] = i < Dl ? __ldg(Gt + (size_t)sel[i] * Nloc) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 32; ++u) {
      const int i = i0 + 4 * u;
      if (i < Dl) A[i * pitch + c] = v[u];
    }
  }
  __syncthreads();
  // softmax over the destinations for source token c of the strip: the column's four threads take every
  // fourth destination; partial maxima and sums meet in shared memory
  float mx = -INFINITY;
#pragma unroll 8
  for (int i = part; i < Dl; i += 4) mx = fmaxf(mx, A[i * pitch + c]);
  red[part * kStrip + c] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red[c], red[kStrip + c]), fmaxf(red[2 * kStrip + c], red[3 * kStrip + c]));
  const float neg_m = -mx * p.scale_log2;
  __syncthreads();
  float sum = 0.f;
#pragma unroll 8
  for (int i = part; i < Dl; i += 4) {
    const float e = ex2f(fmaf(A[i * pitch + c], p.scale_log2, neg_m));
    A[i * pitch + c] = e;
    sum += e;
  }
  red[part * kStrip + c] = sum;
  __syncthreads();
  const float inv = 1.f / ((red[c] + red[kStrip + c]) + (red[2 * kStrip + c] + red[3 * kStrip + c]));
#pragma unroll 8
  for (int i = part; i < Dl; i += 4) A[i * pitch + c] *= inv;
  __syncthreads();
  // this strip's row sums: a warp per destination (two sources per lane, then a fixed tree), sent to every peer
  for (int i = warp; i < Dl; i += 8) {
    float z = A[i * pitch + lane] + A[i * pitch + lane + 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) zpart[rank * Dl + i] = z;
  }
  __syncthreads();
  if (t < 128) {
    for (int q = 0; q < n_cta; ++q) {
      if (q == rank) continue;
      const uint32_t dst = peer_addr(smem_u32(zpart + rank * Dl), (uint32_t)q);
      for (int i = t; i < Dl; i += 128) st_peer_f32(dst + 4u * (uint32_t)i, zpart[rank * Dl + i]);
      mbar_arrive_peer(peer_addr(smem_u32(&bar->z_in), (uint32_t)q));
    }
  }
  const bool got = n_cta == 1 || mbar_wait_cluster(&bar->z_in, 0, dev_status, &bar->abort_flag);
  for (int i = t; i < Dl; i += blockDim.x) {
    float z = 0.f;
    for (int q = 0; q < n_cta; ++q) z += zpart[q * Dl + i];  // strips in rank order, in every CTA
    zinv[i] = (got && z > 0.f) ? 1.f / z : 0.f;               // a row sum that underflowed to 0 gives a zero row
  }
  __syncthreads();
  // A~^T[k][i] = A[i][k] / Z_i as hi + lo planes; consecutive threads write consecutive 16-byte groups of a row
  const int groups = Dl / 8;
  __nv_bfloat16* hi_plane = w + (size_t)tile_b * 2 * Nloc * Dl + (size_t)rank * kStrip * Dl;
  __nv_bfloat16* lo_plane = hi_plane + (size_t)Nloc * Dl;
  for (int q = t; q < kStrip * groups; q += blockDim.x) {
    const int src = q / groups, i0 = (q - src * groups) * 8;
    __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float v = A[(i0 + e) * pitch + src] * zinv[i0 + e];
      hi[e] = __float2bfloat16_rn(v);
      lo[e] = __float2bfloat16_rn(v - __bfloat162float(hi[e]));
    }
    *reinterpret_cast<uint4*>(hi_plane + (size_t)src * Dl + i0) = *reinterpret_cast<const uint4*>(hi);
    *reinterpret_cast<uint4*>(lo_plane + (size_t)src * Dl + i0) = *reinterpret_cast<const uint4*>(lo);
  }
  cluster_sync();  // no CTA's shared memory goes away while a peer could still write to it
}

GParams make_gparams(const Geom& g) {
  GParams p;
  p.P = g.P; p.tiles_x = g.tiles_x; p.th = g.th; p.tw = g.tw; p.Nloc = g.Nloc; p.Dloc = g.Dloc; p.d = g.d;
  p.scale_log2 = g.logit_scale * 1.4426950408889634f;
  return p;
}

}  // namespace

// Shapes and launches the Gram path pays for: bf16, tile-local, transpose unmerge (no second matrix), tiles of 128
// or 256 tokens that are whole TMA boxes, G no larger than the quantised tokens whose place it takes, and so few
// tiles that most SMs are idle while the greedy rounds run.
bool weights_gram_supported(const Geom& g) {
  if (g.f32 || g.global_merge || g.unmerge_mode != TOMA_UNMERGE_TRANSPOSE) return false;
  if (g.Nloc != 128 && g.Nloc != 256) return false;
  if (g.tw > 128 || 128 % g.tw != 0 || g.Nloc / g.tw > 256 || g.th != g.Nloc / g.tw) return false;
  if (g.Dloc % 8 != 0 || g.Dloc < 8 || g.d % 64 != 0) return false;
  if ((size_t)g.Nloc * 4 > (size_t)g.d * 2) return false;
  if (g.Dloc > 256) return false;  // a strip's logits, [D_loc][65] floats, stay far below the shared memory of an SM
  return g.B * g.P <= sm_count() / 2;
}

// G [tile][N_loc][N_loc] fp32 from the raw tokens; to be launched directly behind the greedy kernel.
cudaError_t launch_gram_raw(const Geom& g, const void* x, float* G, uint32_t* dev_status, cudaStream_t s) {
  CUtensorMap ta, tb;
  const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.B};
  const uint64_t strides[3] = {(uint64_t)g.d * 2, (uint64_t)g.W * g.d * 2, (uint64_t)g.tokens_all() * g.d * 2};
  const uint32_t box_a[4] = {64, (uint32_t)g.tw, (uint32_t)(128 / g.tw), 1};
  const uint32_t box_b[4] = {64, (uint32_t)g.tw, (uint32_t)(g.Nloc / g.tw), 1};
  if (!encode_tmap_16bit(&ta, x, 4, dims, strides, box_a) || !encode_tmap_16bit(&tb, x, 4, dims, strides, box_b))
    return cudaErrorInvalidValue;
  const GParams p = make_gparams(g);
  const int ring = kStagesG * (128 * 128 + g.Nloc * 128), staging = 128 * (g.Nloc + 1) * 4;
  const int smem = 1024 + (ring > staging ? ring : staging) + 256;
  static std::atomic<unsigned long long> raised{0};
  cudaError_t e = raise_dynamic_smem(gram_raw_kernel, 227 * 1024, raised);
  if (e != cudaSuccess) return e;
  e = launch_dependent(gram_raw_kernel, dim3(g.B * g.P, g.Nloc / 128), dim3(192), (size_t)smem, s, ta, tb, G, p, dev_status);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_weights_gram(const Geom& g, const float* G, const int32_t* idx, void* w, uint32_t* dev_status, cudaStream_t s) {
  const GParams p = make_gparams(g);
  const int n_cta = g.Nloc / kStrip;
  const size_t smem = ((size_t)g.Dloc * (kStrip + 1) + (size_t)n_cta * g.Dloc + g.Dloc + 4 * kStrip + g.Dloc + 2) * 4 + 64;
  static std::atomic<unsigned long long> raised{0};
  cudaError_t e = raise_dynamic_smem(weights_gram_kernel, 200 * 1024, raised);
  if (e != cudaSuccess) return e;
  e = launch_dependent_cluster(weights_gram_kernel, dim3(g.B * g.P * n_cta), dim3(256), smem, n_cta, s, G, idx, (__nv_bfloat16*)w, p,
                               dev_status);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace toma
