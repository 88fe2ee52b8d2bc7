// Attention core softmax(Q K^T / sqrt(dh)) V (Eq. 1 with tau = 1) on the sm_100a tensor
// cores, bf16 in / bf16 out, fp32 softmax and accumulation.
//
// Work unit = (batch, head, 256 queries) = two 128-row query tiles that share every K/V tile; one
// iteration = one 64-key tile of a unit.  The launch is persistent, one CTA per SM, and the units'
// iterations, laid end to end, are cut into one contiguous span per CTA, so that every CTA runs the
// same number of key tiles whatever the unit count.  A span that covers only part of a unit's keys
// leaves the unnormalised accumulator, the reference maximum and the row sum of its piece in global
// scratch; the warp that arrives last at the (unit, warp) ticket adds the pieces up and writes the
// output rows.  Nobody waits for another CTA.
//
// Inside a CTA (12 warps): warps 0..3 run the online softmax of query tile 0, warps 4..7 that of
// query tile 1 (one thread per query row, straight out of tensor memory), warp 8 feeds Q, K and V
// through TMA rings, one elected thread of warp 9 issues the tcgen05 MMAs (at head_dim 128 those of query tile 0,
// and one of warp 11 those of query tile 1), warp 10 publishes a
// partial first piece (memory fence and tickets, off everybody else's path).
//   S_q,j = Q_q K_j^T      -> tensor memory, two 64-column buffers per query tile.  MMAs issued by
//                             one thread execute in order, so S_q,j+2 is issued right behind the
//                             product that reads P_q,j out of the same buffer, without a round trip
//                             through a barrier: a softmax warp group always finds its next S tile
//                             complete, and the tensor pipe, the two softmax groups and the loads
//                             overlap instead of taking turns.
//   P_q,j = 2^(S*c - m)    -> written back over S_q,j's first 32 columns as bf16 and used as the
//                             A operand (from tensor memory) of  O_q += P_q,j V_j
//   row sums (head_dim 64) -> the B operand of that product is [V_j | 1]: 16 extra columns of ones
//                             accumulate sum_k P_jk behind O in tensor memory: exactly the bf16 P
//                             that multiplies V, so P can be produced by truncation (one
//                             byte-permute per pair, no conversion on the XU pipe) without biasing
//                             the normalised result
//   running maximum        -> O (and the row sums) are rescaled only when the maximum grew by more
//                             than 2^8; the final division by the row sum makes a stale maximum exact
//   exponentials           -> one pair of columns in four (three in eight at head_dim 128) goes through
//                             a degree-3 polynomial on the FMA pipe (relative error 7.5e-5, far below
//                             bf16 resolution of P), the rest through MUFU ex2; the scaling S*c - m and
//                             the polynomial run in packed f32x2 arithmetic (one issue slot for two columns)
// The whole S row of a tile (64 fp32) is fetched with one tensor-memory round trip and kept in
// registers for both the maximum and the exponentials.
// Keys past the sequence end are zero-filled by TMA and masked out; query rows past the end are
// computed on zeros and not written.
#include "attention_core.cuh"
#include "common.cuh"
#include "tc.cuh"

namespace toma {

using namespace tc;
using namespace attn;

namespace {

constexpr int kUM = 2 * kBM;  // queries per work unit
constexpr int kThreads = 384;

template <int DH>
struct AttCfg {
  static constexpr int kStages = 4;                        // K/V ring depth (S runs two tiles ahead of P V)
  static constexpr int kQBufs = DH == 64 ? 2 : 1;          // Q buffers: the next unit's Q lands under this unit's tail
  static constexpr int kChunks = DH / 64;                  // 64-column (128-byte) slabs per row
  static constexpr int kQSlab = kBM * 128;                 // 128 query rows x 128 B
  static constexpr int kQTile = kChunks * kQSlab;          // one query tile
  static constexpr int kQBytes = 2 * kQTile;               // both query tiles of a unit
  static constexpr int kKvSlab = kBN * 128;                // 64 key rows x 128 B
  static constexpr int kKvBytes = kChunks * kKvSlab;       // one K or V tile
  static constexpr bool kSumMma = DH == 64;                // row sums on the tensor pipe, truncated P
  static constexpr int kOnesBytes = kSumMma ? kBN * 128 : 0;  // [64 keys][64] bf16 ones: the N chunk after V in the PV operand
  static constexpr int kOutBytes = 8 * 32 * 128;           // per softmax warp: 32 output rows of one 64-channel slab, staged for a TMA store
  static constexpr int kBarBytes = 512;
  static constexpr int kSmemBytes = 1024 + kQBufs * kQBytes + 2 * kStages * kKvBytes + kOnesBytes + kOutBytes + kBarBytes;
  static constexpr int kTmemCols = 512;
  // Threads that issue MMAs.  With two, each query tile has its own (on different schedulers): neither waits behind
  // the other tile's barrier.  Timed: 2-3.5 % faster at head_dim 128, 0-1.4 % slower at head_dim 64.
  static constexpr int kIssuers = DH == 128 ? 2 : 1;
  // S buffer (q, b) at column (2 q + b) * 64; O_q (and, behind it, the row sums) from column 256
  static constexpr int kColS = 0, kColO = 256, kOStride = DH == 64 ? 96 : 128;
};

struct Barriers {
  uint64_t q_full[2], q_empty[2];     // per piece: Q landed / every S MMA of the piece has read Q
  uint64_t k_full[4], kv_empty[4];    // per tile: K and V landed / every MMA that reads them is done
  uint64_t s_full[2][2], p_full[2][2];  // per tile and query tile: S ready for the softmax / P ready for the PV MMAs
  uint64_t o_done[2], o_free[2];      // per piece and query tile: accumulator complete / epilogue has read it
  uint64_t pub_ready, pub_done;       // first partial piece: written by the softmax warps / published, tickets drawn
  uint32_t first_ticket[8];           // per softmax warp: ticket its first (partial) piece drew
  uint32_t others_done;               // set by the publisher when the span's last unit has all its other pieces in scratch
  uint32_t poll_stop[2];              // set by each softmax group when the answer is no longer needed
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Barriers) <= 512, "barrier block outgrew its reservation");

constexpr int kSnapTiles = 2;
constexpr int kMaxCtas = 160;  // scratch and the span table are sized for this many persistent CTAs (ids fit a byte)

// The iterations [0, T) are cut into G contiguous spans, CTA g running [bounds[g], bounds[g + 1]).
// With whole units every bound is a multiple of nblk (no scratch traffic), which wins when the unit
// count happens to fill the CTAs evenly; otherwise the spans are cut at single key tiles so that the
// longest span is as short as possible when every piece is charged its pipeline drain and epilogue
// (plan_spans): a piece of one or two tiles costs its CTA more than the tiles it moves are worth.
struct Spans {
  int T, G, nblk, split;
  int bounds[kMaxCtas + 1];
  // Lowest and highest CTA among those whose spans hold key tiles of the unit CTA g's span starts in ([0][g])
  // and of the unit it ends in ([1][g]): the only units a CTA can share.  Filled in by the host, so that the
  // kernel does not search the bounds at the end of a piece.
  uint8_t unit_lo[2][kMaxCtas], unit_hi[2][kMaxCtas];
  __host__ __device__ int bound(int g) const { return bounds[g]; }
  // the CTA whose span holds iteration `it`
  __host__ __device__ int owner(int it) const {
    int lo = 0, hi = G - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (bounds[mid] <= it) lo = mid;
      else hi = mid - 1;
    }
    return lo;
  }
};

// One piece = the part of a span inside one unit: key tiles [k0, k0 + cnt) of unit u.
struct Piece {
  int u, k0, cnt;
};
__device__ __forceinline__ Piece piece_at(int it, int it_end, int nblk) {
  Piece p;
  p.u = it / nblk;
  p.k0 = it - p.u * nblk;
  const int left = it_end - it;
  p.cnt = left < nblk - p.k0 ? left : nblk - p.k0;
  return p;
}

// A position in the CTA's span for the single-thread roles: `n` counts key tiles across pieces (ring
// slots, S buffers and their barrier phases follow n), `pc` counts pieces (phases of the per-piece
// barriers), `j` is the tile inside the current piece of `cnt` tiles.
struct Cursor {
  int it, it_end, nblk, j, cnt, pc, n;
  __device__ __forceinline__ void load() {
    const int left = it_end - it, in_unit = nblk - it % nblk;
    cnt = left < in_unit ? left : in_unit;
  }
  __device__ __forceinline__ void init(int b, int e, int nb) {
    it = b, it_end = e, nblk = nb, j = 0, pc = 0, n = 0;
    load();
  }
  __device__ __forceinline__ bool valid() const { return it < it_end; }
  __device__ __forceinline__ bool last_of_piece() const { return j + 1 == cnt; }
  __device__ __forceinline__ void next() {
    ++n;
    if (++j == cnt) {
      it += cnt, ++pc, j = 0;
      load();
    }
  }
};

// Scratch of one piece: O as [DH / 4][256 rows] float4, then m[256], l[256].
template <int DH>
__host__ __device__ constexpr size_t piece_floats() { return (size_t)kUM * DH + 2 * kUM; }

// Where the output rows of unit u start for query row `row` (0..255) of the unit (nullptr past the sequence end).
template <int DH>
__device__ __forceinline__ __nv_bfloat16* out_row(__nv_bfloat16* o, int u, int row, int L, int heads) {
  const int nq = (L + kUM - 1) / kUM;
  const int bh = u / nq, qi = (u - bh * nq) * kUM + row, b = bh / heads, h = bh - b * heads;
  if (qi >= L) return nullptr;
  return o + ((size_t)b * L + qi) * ((size_t)heads * DH) + (size_t)h * DH;
}

// Scratch slot of the piece of unit u that CTA g left: its first piece sits in slot 0, a later
// partial piece (necessarily its last) in slot 1.
template <int DH>
__device__ __forceinline__ const float* slot_of(const float* pieces, const Spans& sp, int g, int u) {
  const int first_unit = sp.bound(g) / sp.nblk;
  return pieces + (size_t)(2 * g + (u > first_unit ? 1 : 0)) * piece_floats<DH>();
}

// Adds up the pieces of one query row of unit u, left by CTAs g_first..g_last:
//   O = sum_i 2^(m_i - M) O_i / sum_i 2^(m_i - M) l_i,  M = max_i m_i  (m in the log2 domain).
// Contributors are taken two at a time so that their loads are in flight together, and summed in
// ascending CTA order with one fused multiply-add each, starting from zero: finish_piece's direct
// path follows the same order, so the result does not depend on which path a launch takes.  Loads bypass L1: the pieces were written by other SMs during this launch.
template <int DH>
__device__ __noinline__ void combine_rows(const float* pieces, const Spans& sp, int u, int g_first, int g_last, int row,
                                          __nv_bfloat16* dst) {
  constexpr size_t kM = (size_t)kUM * DH, kL = (size_t)kUM * DH + kUM;
  float M = -INFINITY;
  for (int g = g_first; g <= g_last; g += 2) {
    const float* sa = slot_of<DH>(pieces, sp, g, u);
    const float* sb = g < g_last ? slot_of<DH>(pieces, sp, g + 1, u) : sa;
    M = max3(M, __ldcg(sa + kM + row), __ldcg(sb + kM + row));
  }
#pragma unroll 1
  for (int half = 0; half < DH / 64; ++half) {  // 64 accumulator columns at a time
    float denom = 0.f;
    float acc[64];
#pragma unroll
    for (int e = 0; e < 64; ++e) acc[e] = 0.f;
    for (int g = g_first; g <= g_last; g += 2) {
      const float* sa = slot_of<DH>(pieces, sp, g, u);
      const float* sb = g < g_last ? slot_of<DH>(pieces, sp, g + 1, u) : sa;
      const float ma = __ldcg(sa + kM + row), la = __ldcg(sa + kL + row);
      const float mb = __ldcg(sb + kM + row), lb = __ldcg(sb + kL + row);
      const float wa = ex2_mufu(ma - M), wb = g < g_last ? ex2_mufu(mb - M) : 0.f;
      denom = fmaf(wb, lb, fmaf(wa, la, denom));
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float4 va[8], vb[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          va[q] = __ldcg(reinterpret_cast<const float4*>(sa) + (size_t)(half * 16 + c * 8 + q) * kUM + row);
          vb[q] = __ldcg(reinterpret_cast<const float4*>(sb) + (size_t)(half * 16 + c * 8 + q) * kUM + row);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          float* a4 = &acc[c * 32 + 4 * q];
          a4[0] = fmaf(wb, vb[q].x, fmaf(wa, va[q].x, a4[0]));
          a4[1] = fmaf(wb, vb[q].y, fmaf(wa, va[q].y, a4[1]));
          a4[2] = fmaf(wb, vb[q].z, fmaf(wa, va[q].z, a4[2]));
          a4[3] = fmaf(wb, vb[q].w, fmaf(wa, va[q].w, a4[3]));
        }
      }
    }
    if (!dst) continue;
    const float inv = 1.f / denom;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      uint32_t r[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(acc[c * 32 + e]);
      store_row32(dst + half * 64 + c * 32, r, inv);
    }
  }
}

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void st_release_cta(uint32_t* smem_word, uint32_t v) {
  asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(smem_word)), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_cta(const uint32_t* smem_word) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(smem_word)) : "memory");
  return v;
}

// Publishes this warp's 32 rows of a piece and takes the (unit, warp) ticket.  Returns the number
// of contributors that had taken it before.  Called by whole warps only.
__device__ __forceinline__ uint32_t take_ticket(uint32_t* ticket, int lane) {
  __threadfence();
  __syncwarp();
  uint32_t t = 0;
  if (lane == 0) t = atomicAdd(ticket, 1u);
  return __shfl_sync(0xffffffffu, t, 0);
}

// The per-thread view of a softmax thread: its query tile, its row in the unit, its accumulator.
struct Row {
  int q;        // query tile (softmax warp group) 0 or 1
  int warp;     // softmax warp 0..7 = ticket column
  int lane;
  int row;      // query row inside the unit, 0..255
  uint32_t ob;  // tensor-memory address of this row's accumulator
};
// Where a softmax warp stages its output rows, and the map they are stored through: kept out of Row (the softmax
// loop holds a Row in registers) and derived where a piece ends.
struct OutStage {
  uint8_t* stage;           // this warp's 4 KB of the output staging area (it lies right below the barriers)
  const CUtensorMap* tm_o;  // output as (channel, token, batch), box = 64 channels x 32 tokens
};
template <int DH>
__device__ __forceinline__ OutStage out_stage(const void* bar, int warp, const CUtensorMap* tm_o) {
  return OutStage{const_cast<uint8_t*>(reinterpret_cast<const uint8_t*>(bar)) - AttCfg<DH>::kOutBytes + warp * 4096, tm_o};
}

// Output rows leave through shared memory: a thread puts 32 channels of its row (scaled, bf16) into its warp's
// staged slab (64 channels x 32 rows, 128-byte swizzled = the output map's box), and when a slab is complete the
// warp stores it with one TMA store - whole lines instead of 16-byte stores to 32 different rows per warp
// instruction.  Rows past the end of the sequence are clipped by the store.
__device__ __forceinline__ void stage_half(const OutStage& os, int lane, int half, const uint32_t (&r)[32], float inv) {
#pragma unroll
  for (int e = 0; e < 32; e += 8) {
    uint4 v;
    v.x = pack_bf16_rn(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
    v.y = pack_bf16_rn(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
    v.z = pack_bf16_rn(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
    v.w = pack_bf16_rn(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
    *reinterpret_cast<uint4*>(os.stage + sw128_offset(lane, half * 4 + (e >> 3))) = v;
  }
}
// The same for 16 channels (quarter 0..3 of the slab's 64).
__device__ __forceinline__ void stage_quarter(const OutStage& os, int lane, int quarter, const uint32_t (&r)[16], float inv) {
#pragma unroll
  for (int e = 0; e < 16; e += 8) {
    uint4 v;
    v.x = pack_bf16_rn(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
    v.y = pack_bf16_rn(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
    v.z = pack_bf16_rn(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
    v.w = pack_bf16_rn(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
    *reinterpret_cast<uint4*>(os.stage + sw128_offset(lane, quarter * 2 + (e >> 3))) = v;
  }
}
// Whole warp.  (ch0, row0, b): first channel of the slab, first token of the warp's 32 rows, batch item.
__device__ __forceinline__ void flush_slab(const OutStage& os, int lane, int ch0, int row0, int b, int L) {
  fence_proxy_async();  // the staged rows are read by the TMA engine
  __syncwarp();
  if (lane == 0 && row0 < L) {
    tma_store_3d(os.tm_o, os.stage, ch0, row0, b);
    tma_store_commit();
    tma_store_wait_read();  // the slab is staged again right away
  }
  __syncwarp();
}
// Batch item, first channel and first token of the 32 rows that warp t.warp holds of unit u.
template <int DH>
__device__ __forceinline__ void warp_rows_of(int u, const Row& t, int L, int heads, int& b, int& ch0, int& row0) {
  const int nq = (L + kUM - 1) / kUM;
  const int bh = u / nq;
  b = bh / heads;
  ch0 = (bh - b * heads) * DH;
  row0 = (u - bh * nq) * kUM + (t.row & ~31);
}

// End of a piece that covers all keys of its unit (the only kind when units are kept whole), run by
// the softmax warps: wait for the accumulator, normalise, write the rows out.  Returns false when
// the wait ran out.
template <int DH>
__device__ __forceinline__ bool finish_whole(const Row& t, Barriers* bar, int unit, int pc, float l, const CUtensorMap* tm_o, int L,
                                             int heads, uint32_t* dev_status) {
  using C = AttCfg<DH>;
  if (!mbar_wait(&bar->o_done[t.q], pc & 1, dev_status, &bar->abort_flag)) return false;
  tc_fence_after();
  if (C::kSumMma) {
    uint32_t rs[16];
    tmem_ld16(t.ob + DH, rs);
    tmem_wait_ld();
    l = __uint_as_float(rs[0]);
  }
  int b, ch0, row0;
  warp_rows_of<DH>(unit, t, L, heads, b, ch0, row0);
  const OutStage os = out_stage<DH>(bar, t.warp, tm_o);
  const float inv = 1.f / l;
#pragma unroll
  for (int c = 0; c < DH / 32; ++c) {
    uint32_t r[32];
    tmem_ld32(t.ob + c * 32, r);
    tmem_wait_ld();
    stage_half(os, t.lane, c & 1, r, inv);
    if (c & 1) flush_slab(os, t.lane, ch0 + (c >> 1) * 64, row0, b, L);
  }
  tc_fence_before();
  __syncwarp();
  if (t.lane == 0) mbar_arrive(&bar->o_free[t.q]);  // the next piece's first PV product may overwrite the accumulator
  return true;
}

// End of a piece that covers only part of its unit's keys, run by the softmax warps:
//   - the last piece of the CTA's span, when the unit's only other contributor has already
//     published (it ran at the start of its own span, so it normally has), is added to that
//     contributor's piece straight from tensor memory and written out: nothing of it goes through
//     scratch, and the other piece is fetched while the last MMAs drain;
//   - any other piece is left in scratch with its reference maximum and row sum and a (unit, warp)
//     ticket is drawn; the warp that draws a unit's last ticket adds its pieces up.  A last piece
//     does that here; a first piece, with more of the span to come, hands the fence and the
//     tickets' round trips to the publisher thread and looks at the outcome in settle_first_piece.
// Every decision that ends in a warp-wide operation is taken once per warp (lane 0 reads, the warp
// gets the value by shuffle), so a warp always goes one way as a whole.
// Out of line (it runs at most twice per CTA and is register-hungry).  Returns false when the wait
// ran out.
template <int DH>
__device__ __noinline__ bool finish_partial(Row t, Barriers* bar, Piece p, int pc, bool last_of_span, float m_used, float l,
                                            __nv_bfloat16* o, const CUtensorMap* tm_o, int L, int heads, const Spans& sp,
                                            uint32_t* tickets, float* pieces, uint32_t* dev_status) {
  using C = AttCfg<DH>;
  constexpr size_t kM = (size_t)kUM * DH, kL = (size_t)kUM * DH + kUM;
  const int row = t.row, lane = t.lane;
  uint32_t* ticket = tickets + (size_t)p.u * 8 + t.warp;
  // a partial piece lies in the unit the span starts in or in the one it ends in
  const int which = p.u == sp.bound(blockIdx.x) / sp.nblk ? 0 : 1;
  const int g_first = sp.unit_lo[which][blockIdx.x], g_last = sp.unit_hi[which][blockIdx.x];
  bool own_first = false;  // this CTA is the lower of the two contributors
  // The direct path comes in two forms.  The wide one holds 64 columns of the other piece in registers (the
  // function then spills); the lean one takes 16 columns at a time with the next 16 on their way.  Timed as a
  // whole, the kernel is 3-4 % faster with the lean form at head_dim 128 and 5-7 % slower at head_dim 64, where
  // the register allocation of the tile loop changes with this function's needs: each keeps the form that wins.
  constexpr bool kLean = DH == 128;
  const float* other = nullptr;
  float m_o = 0.f, l_o = 0.f;
  float4 vo[kLean ? 4 : 16];
  // the publisher warp watches the tickets of the span's last unit; its answer carries the
  // acquire that orders the loads below after the other contributor's writes
  uint32_t others = 0;
  if (last_of_span && g_last == g_first + 1) {
    if (lane == 0) others = ld_acquire_cta(&bar->others_done);
    __syncwarp();
    others = __shfl_sync(0xffffffffu, others, 0);
  }
  const bool direct = others == 1u;
  if (last_of_span && (row & (kBM - 1)) == 0) *(volatile uint32_t*)&bar->poll_stop[t.q] = 1u;
  if (direct) {
    own_first = (int)blockIdx.x == g_first;
    other = slot_of<DH>(pieces, sp, own_first ? g_last : g_first, p.u);
    m_o = __ldcg(other + kM + row);
    l_o = __ldcg(other + kL + row);
#pragma unroll
    for (int q = 0; q < (kLean ? 4 : 16); ++q) vo[q] = __ldcg(reinterpret_cast<const float4*>(other) + (size_t)q * kUM + row);
  }
  if (!mbar_wait(&bar->o_done[t.q], pc & 1, dev_status, &bar->abort_flag)) return false;
  tc_fence_after();
  if (C::kSumMma) {
    uint32_t rs[16];
    tmem_ld16(t.ob + DH, rs);
    tmem_wait_ld();
    l = __uint_as_float(rs[0]);
  }
  __nv_bfloat16* dst = out_row<DH>(o, p.u, row, L, heads);
  int b_item, ch0, row0;
  warp_rows_of<DH>(p.u, t, L, heads, b_item, ch0, row0);
  const OutStage os = out_stage<DH>(bar, t.warp, tm_o);
  float* slot = pieces + (size_t)(2 * blockIdx.x + (pc > 0 ? 1 : 0)) * piece_floats<DH>();
  float w_own = 1.f, w_o = 0.f, inv = 1.f;
  if (direct) {
    const float M = fmaxf(m_used, m_o);
    w_own = ex2_mufu(m_used - M);
    w_o = ex2_mufu(m_o - M);
    inv = 1.f / (own_first ? fmaf(w_o, l_o, w_own * l) : fmaf(w_own, l, w_o * l_o));
  }
  // rows of the piece into its scratch slot (32 columns at a time)
  auto to_scratch = [&](int c, const uint32_t (&r)[32]) {
#pragma unroll
    for (int e = 0; e < 32; e += 4)
      reinterpret_cast<float4*>(slot)[(size_t)(c * 8 + (e >> 2)) * kUM + row] =
          make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
  };
  if constexpr (kLean) {
    if (direct) {
#pragma unroll
      for (int c = 0; c < DH / 16; ++c) {
        float4 vc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) vc[q] = vo[q];
        if (c + 1 < DH / 16) {
#pragma unroll
          for (int q = 0; q < 4; ++q) vo[q] = __ldcg(reinterpret_cast<const float4*>(other) + (size_t)((c + 1) * 4 + q) * kUM + row);
        }
        uint32_t r[16];
        tmem_ld16(t.ob + c * 16, r);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float vv[4] = {vc[q].x, vc[q].y, vc[q].z, vc[q].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float own = __uint_as_float(r[4 * q + e]);
            r[4 * q + e] = __float_as_uint(own_first ? fmaf(w_o, vv[e], w_own * own) : fmaf(w_own, own, w_o * vv[e]));
          }
        }
        stage_quarter(os, t.lane, c & 3, r, inv);
        if ((c & 3) == 3) flush_slab(os, t.lane, ch0 + (c >> 2) * 64, row0, b_item, L);
      }
    } else {
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(t.ob + c * 32, r);
        tmem_wait_ld();
        to_scratch(c, r);
      }
    }
  } else {
#pragma unroll
    for (int c = 0; c < DH / 32; ++c) {
      uint32_t r[32];
      tmem_ld32(t.ob + c * 32, r);
      tmem_wait_ld();
      if (direct) {
        if (c > 0 && (c & 1) == 0) {  // next 64 columns of the other piece
#pragma unroll
          for (int q = 0; q < 16; ++q) vo[q] = __ldcg(reinterpret_cast<const float4*>(other) + (size_t)(c * 8 + q) * kUM + row);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 v = vo[(c & 1) * 8 + q];
          const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float own = __uint_as_float(r[4 * q + e]);
            r[4 * q + e] = __float_as_uint(own_first ? fmaf(w_o, vv[e], w_own * own) : fmaf(w_own, own, w_o * vv[e]));
          }
        }
        stage_half(os, t.lane, c & 1, r, inv);
        if (c & 1) flush_slab(os, t.lane, ch0 + (c >> 1) * 64, row0, b_item, L);
      } else {
        to_scratch(c, r);
      }
    }
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(&bar->o_free[t.q]);  // the next piece's first PV product may overwrite the accumulator
  if (direct) return true;
  slot[kM + row] = m_used;
  slot[kL + row] = l;
  if (!last_of_span) {  // the publisher thread fences, draws the tickets and leaves them for settle_first_piece
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar->pub_ready);
  } else if (take_ticket(ticket, lane) == (uint32_t)(g_last - g_first)) {
    __threadfence();
    combine_rows<DH>(pieces, sp, p.u, g_first, g_last, row, dst);
  }
  return true;
}

// End of a CTA's span: if its first piece was partial and took the unit's last ticket (the other
// contributors, which run that unit at the end of their spans, are normally later), add the
// unit's pieces up now.
template <int DH>
__device__ __noinline__ void settle_first_piece(Barriers* bar, int it_begin, int it_end, Row t, __nv_bfloat16* o, int L,
                                                int heads, const Spans& sp, const float* pieces, uint32_t* dev_status) {
  const int nblk = sp.nblk, u = it_begin / nblk;
  const bool first_partial = it_begin > u * nblk || it_end < (u + 1) * nblk;
  if (!first_partial || it_end <= (u + 1) * nblk) return;  // whole, or also the span's last piece: settled already
  const int g_first = sp.unit_lo[0][blockIdx.x], g_last = sp.unit_hi[0][blockIdx.x];
  if (!mbar_wait(&bar->pub_done, 0, dev_status, &bar->abort_flag)) return;
  if (bar->first_ticket[t.warp] != (uint32_t)(g_last - g_first)) return;
  __threadfence();
  combine_rows<DH>(pieces, sp, u, g_first, g_last, t.row, out_row<DH>(o, u, t.row, L, heads));
}

// The ragged last key tile of a sequence: out of line, so that the hot loop holds one copy of the
// softmax code.
template <int DH>
__device__ __noinline__ bool softmax_tile_ragged(uint32_t sb, uint32_t ob, float scale_log2, int valid, int j, float& m_used,
                                                 float& l, uint64_t* pv_done, uint32_t pv_parity, uint32_t* dev_status,
                                                 volatile int* abort_flag) {
  return softmax_tile<DH, AttCfg<DH>::kSumMma, true>(sb, ob, scale_log2, valid, j, m_used, l, pv_done, pv_parity, dev_status, abort_flag);
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                    __nv_bfloat16* __restrict__ o, int L, int heads,
                    float scale_log2, const __grid_constant__ Spans sp, uint32_t* __restrict__ tickets, float* __restrict__ pieces,
                    uint32_t* dev_status) {
  using C = AttCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + C::kQBufs * C::kQBytes;
  uint8_t* sV = sK + C::kStages * C::kKvBytes;
  uint8_t* sOnes = sV + C::kStages * C::kKvBytes;
  uint8_t* sOut = sOnes + C::kOnesBytes;
  Barriers* bar = reinterpret_cast<Barriers*>(sOut + C::kOutBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nblk = sp.nblk;
  const int nq = (L + kUM - 1) / kUM;  // units per (batch, head)
  const int it_begin = sp.bound(blockIdx.x), it_end = sp.bound(blockIdx.x + 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->q_full[s], 1);
      mbar_init(&bar->q_empty[s], C::kIssuers);
      mbar_init(&bar->o_done[s], 1);
      mbar_init(&bar->o_free[s], 4);  // one arrival per softmax warp of the group
      for (int b = 0; b < 2; ++b) {
        mbar_init(&bar->s_full[s][b], 1);
        mbar_init(&bar->p_full[s][b], 4);
      }
      bar->poll_stop[s] = 0;
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->kv_empty[s], C::kIssuers);
    }
    mbar_init(&bar->pub_ready, 8);
    mbar_init(&bar->pub_done, 1);
    bar->others_done = 0;
    bar->abort_flag = 0;
    mbar_fence_init();
  }
  if (C::kSumMma) {  // bf16 1.0 everywhere: the layout's swizzle is irrelevant for a constant tile
    for (int e = threadIdx.x; e < C::kOnesBytes / 4; e += blockDim.x) reinterpret_cast<uint32_t*>(sOnes)[e] = 0x3F803F80u;
    fence_proxy_async();
  }
  if (threadIdx.x == 256) {  // descriptor fetches overlap the previous kernel's tail
    prefetch_tmap(&tm_q);
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
    prefetch_tmap(&tm_o);
  }
  dependency_wait();
  if (threadIdx.x == 0) release_dependents();
  if (warp == 9) tmem_alloc(&bar->tmem_base, C::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  volatile int* abort_flag = &bar->abort_flag;

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      Cursor c;
      for (c.init(it_begin, it_end, nblk); c.valid(); c.next()) {
        if (c.j == 0) {
          const int u = c.it / nblk;
          const int bh = u / nq, q0 = (u - bh * nq) * kUM, b = bh / heads, h = bh - b * heads;
          const int qb = c.pc % C::kQBufs;
          // a Q buffer is free once the S MMAs of the piece that used it have read it
          if (c.pc >= C::kQBufs && !mbar_wait(&bar->q_empty[qb], ((c.pc / C::kQBufs) - 1) & 1, dev_status, abort_flag)) break;
          mbar_expect_tx(&bar->q_full[qb], C::kQBytes);
          for (int t = 0; t < 2; ++t)
            for (int ch = 0; ch < C::kChunks; ++ch)
              tma_load_3d(sQ + qb * C::kQBytes + t * C::kQTile + ch * C::kQSlab, &tm_q, &bar->q_full[qb], h * DH + ch * 64,
                          q0 + t * kBM, b);
        }
        const int u = c.it / nblk, k0 = c.it - u * nblk;
        const int bh = u / nq, b = bh / heads, h = bh - b * heads;
        const int s = c.n % C::kStages;
        if (c.n >= C::kStages && !mbar_wait(&bar->kv_empty[s], ((c.n / C::kStages) - 1) & 1, dev_status, abort_flag)) break;
        const int key0 = (k0 + c.j) * kBN;
        mbar_expect_tx(&bar->k_full[s], 2 * C::kKvBytes);  // K and V of a tile arrive under one barrier
        for (int ch = 0; ch < C::kChunks; ++ch)
          tma_load_3d(sK + s * C::kKvBytes + ch * C::kKvSlab, &tm_k, &bar->k_full[s], h * DH + ch * 64, key0, b);
        for (int ch = 0; ch < C::kChunks; ++ch)
          tma_load_3d(sV + s * C::kKvBytes + ch * C::kKvSlab, &tm_v, &bar->k_full[s], h * DH + ch * 64, key0, b);
      }
    }
  } else if (warp == 9 || (warp == 11 && C::kIssuers == 2)) {
    // ------------------------------------------------------------------ MMA issuer(s)
    // A thread's MMAs execute in the order it issues them: the S product of tile n+2 goes into the buffer whose
    // P the PV product of tile n, issued just before by the same thread, still reads.  The two query tiles'
    // products are independent of each other: one thread issues both, or each tile has its own thread
    // (query tiles [q_lo, q_hi) here); the barriers that both tiles' products free count one arrival per thread.
    const int q_lo = C::kIssuers == 2 && warp == 11 ? 1 : 0, q_hi = C::kIssuers == 2 && warp == 9 ? 1 : 2;
    if (elect_one()) {
      constexpr uint32_t idesc_s = idesc_f16(kFmtBF16, kFmtBF16, false, false, kBM, kBN);
      // With row sums on the tensor pipe the B operand is [V | ones]: N = DH + 16, the 16 extra
      // columns come from a constant slab of ones placed one "leading byte offset" after V's slab,
      // so one MMA per 16 keys updates O and the row sums (which sit right behind O in tensor memory).
      constexpr uint32_t idesc_o = idesc_f16(kFmtBF16, kFmtBF16, false, true, kBM, C::kSumMma ? DH + 16 : DH);
      // Descriptors are built once and advanced by adding a constant to the 14-bit start-address
      // field (no carry: all tiles live below 256 KB).
      const uint64_t q_desc0 = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(sK), 16, 1024);
      const uint32_t v_addr0 = smem_u32(sV), ones_addr = smem_u32(sOnes);
      Cursor cs, cp;  // the S products run two tiles ahead of the PV products
      cs.init(it_begin, it_end, nblk);
      cp.init(it_begin, it_end, nblk);
      bool ok = true;
      // Q of the piece and K of the tile that `cs` points at have landed
      auto s_inputs = [&]() -> bool {
        if (cs.j == 0 && !mbar_wait(&bar->q_full[cs.pc % C::kQBufs], (cs.pc / C::kQBufs) & 1, dev_status, abort_flag)) return false;
        return mbar_wait(&bar->k_full[cs.n % C::kStages], (cs.n / C::kStages) & 1, dev_status, abort_flag);
      };
      auto issue_s = [&](int q) {
        const int s = cs.n % C::kStages, b = cs.n & 1, qb = cs.pc % C::kQBufs;
        const uint64_t qd = q_desc0 + (uint64_t)((qb * C::kQBytes + q * C::kQTile) >> 4);
        const uint64_t kd = k_desc0 + (uint64_t)((s * C::kKvBytes) >> 4);
        const uint32_t t_s = tmem + C::kColS + (2 * q + b) * kBN;
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint64_t qoff = (uint64_t)(((kk >> 2) * C::kQSlab + (kk & 3) * 32) >> 4);
          const uint64_t koff = (uint64_t)(((kk >> 2) * C::kKvSlab + (kk & 3) * 32) >> 4);
          mma_ss(t_s, qd + qoff, kd + koff, idesc_s, kk > 0);
        }
        mma_commit(&bar->s_full[q][b]);
      };
      for (int pre = 0; pre < 2 && ok && cs.valid(); ++pre) {
        ok = s_inputs();
        if (!ok) break;
        tc_fence_after();
        for (int q = q_lo; q < q_hi; ++q) issue_s(q);
        if (cs.last_of_piece()) mma_commit(&bar->q_empty[cs.pc % C::kQBufs]);
        cs.next();
      }
      while (ok && cp.valid()) {
        const int s = cp.n % C::kStages, b = cp.n & 1;
        const bool more = cs.valid();
        const uint32_t va = v_addr0 + s * C::kKvBytes;
        const uint64_t vd = smem_desc_sw128(va, C::kSumMma ? ones_addr - va : (uint32_t)C::kKvSlab, 1024);
#pragma unroll
        for (int q = q_lo; q < q_hi; ++q) {
          // P ready implies that the K/V tile has landed
          if (!mbar_wait(&bar->p_full[q][b], (cp.n >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
          // the first product of a piece overwrites the accumulator the previous epilogue reads
          if (cp.j == 0 && cp.pc > 0 && !mbar_wait(&bar->o_free[q], (cp.pc - 1) & 1, dev_status, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t t_o = tmem + C::kColO + q * C::kOStride;
          const uint32_t t_p = tmem + C::kColS + (2 * q + b) * kBN;
#pragma unroll
          for (int kk = 0; kk < kBN / 16; ++kk)  // 16 keys per MMA: 8 packed columns of P, 16 rows of V
            mma_ts(t_o, t_p + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o, cp.j > 0 || kk > 0);
          // One phase per piece: the next piece's products wait for o_free, which the epilogue gives
          // only after it has seen this phase, so a waiter is never two phases behind.
          if (cp.last_of_piece()) mma_commit(&bar->o_done[q]);
          if (q == q_hi - 1) mma_commit(&bar->kv_empty[s]);  // frees the K/V slot; also "PV of this tile has landed" for a rescale
          if (more) {
            if (q == q_lo) {
              ok = s_inputs();
              if (!ok) break;
              tc_fence_after();
            }
            issue_s(q);
          }
        }
        if (!ok) break;
        if (more) {
          if (cs.last_of_piece()) mma_commit(&bar->q_empty[cs.pc % C::kQBufs]);
          cs.next();
        }
        cp.next();
      }
    }
  } else if (warp == 10) {
    // ------------------------------------------------------------------ publisher
    if (lane == 0) {
      // When the span's first piece is partial and more pieces follow, make that piece
      // visible to the other CTAs and draw its eight tickets here, off the softmax warps' path.
      const int u = it_begin / nblk;
      const bool early = (it_begin > u * nblk || it_end < (u + 1) * nblk) && it_end > (u + 1) * nblk;
      if (early && mbar_wait(&bar->pub_ready, 0, dev_status, abort_flag)) {
        __threadfence();
        uint32_t t[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) t[w] = atomicAdd(&tickets[(size_t)u * 8 + w], 1u);
#pragma unroll
        for (int w = 0; w < 8; ++w) bar->first_ticket[w] = t[w];
        mbar_arrive(&bar->pub_done);
      }
      // When the span ends inside a unit that one other CTA shares, that CTA ran its part at the
      // start of its span and has normally published it long since.  Watch its eight tickets (acquire)
      // and leave the answer in shared memory for the softmax warps: they add the two pieces up
      // straight from tensor memory if the answer is there when their last piece ends, and go
      // through scratch and tickets otherwise.  Polling keeps the ticket out of their registers.
      const int ul = (it_end - 1) / nblk;
      if (it_end < (ul + 1) * nblk && sp.unit_hi[1][blockIdx.x] == sp.unit_lo[1][blockIdx.x] + 1) {
        const uint32_t* tk = tickets + (size_t)ul * 8;
        for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
          if ((*(volatile uint32_t*)&bar->poll_stop[0] && *(volatile uint32_t*)&bar->poll_stop[1]) || *abort_flag) break;
          bool all = true;
#pragma unroll
          for (int w = 0; w < 8; ++w) all = all && ld_acquire_gpu(tk + w) == 1u;
          if (all) {
            st_release_cta(&bar->others_done, 1u);
            break;
          }
          __nanosleep(500);
        }
      }
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------------ softmax / correction / epilogue
    Row t;
    t.q = warp >> 2, t.warp = warp, t.lane = lane;
    t.row = warp * 32 + lane;  // query row inside the unit; (warp & 3) * 32 + lane is its tensor-memory lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    t.ob = tmem + lane_addr + C::kColO + t.q * C::kOStride;
    bool ok = true;
    int n = 0, pc = 0;
    for (int it = it_begin; ok && it < it_end; ++pc) {
      const Piece p = piece_at(it, it_end, nblk);
      it += p.cnt;
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < p.cnt; ++j, ++n) {
        const int b = n & 1;
        const uint32_t sb = tmem + lane_addr + C::kColS + (2 * t.q + b) * kBN;
        if (!mbar_wait(&bar->s_full[t.q][b], (n >> 1) & 1, dev_status, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int valid = L - (p.k0 + j) * kBN;  // keys of this tile inside the sequence (>= 64: all)
        uint64_t* pvb = &bar->kv_empty[(n + C::kStages - 1) % C::kStages];  // barrier the previous tile's PV commits to
        const uint32_t pvp = (uint32_t)(((n - 1) / C::kStages) & 1);
        if (valid >= kBN) ok = softmax_tile<DH, C::kSumMma, false>(sb, t.ob, scale_log2, kBN, j, m_used, l, pvb, pvp, dev_status, abort_flag);
        else ok = softmax_tile_ragged<DH>(sb, t.ob, scale_log2, valid, j, m_used, l, pvb, pvp, dev_status, abort_flag);
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar->p_full[t.q][b]);
      }
      if (!ok) break;
      if (p.cnt == nblk) ok = finish_whole<DH>(t, bar, p.u, pc, l, &tm_o, L, heads, dev_status);
      else ok = finish_partial<DH>(t, bar, p, pc, it >= it_end, m_used, l, o, &tm_o, L, heads, sp, tickets, pieces, dev_status);
    }
    if (ok) settle_first_piece<DH>(bar, it_begin, it_end, t, o, L, heads, sp, pieces, dev_status);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, C::kTmemCols);
  }
}

size_t ticket_bytes(int B, int L, int heads) {
  const size_t units = (size_t)B * heads * ((L + kUM - 1) / kUM);
  return (units * 8 * sizeof(uint32_t) + 255) & ~(size_t)255;
}

int max_ctas() {
  const int sms = sm_count();
  int G = sms < kMaxCtas ? sms : kMaxCtas;
  const int v = g_tune_attention_ctas.load(std::memory_order_relaxed);  // test-only override
  if (v >= 1 && v <= kMaxCtas) G = v;
  return G;
}

// Key tiles a split costs a CTA, in units of one tile's time: writing, publishing and adding up the
// partial results at the end of its span.
constexpr int kSplitCostTiles = 4;

// What a piece costs its CTA beyond its key tiles, in half tiles: the pipeline drains, the accumulator is read
// out and (partial pieces) goes through scratch, tickets and the addition of the unit's pieces.
constexpr int kPieceCostWhole = 4, kPieceCostPartial = 8;

// The farthest end of a span that starts at iteration `start` and costs at most C half tiles
// (2 per key tile plus the piece costs above); `start` itself when not even one tile fits.
int span_end(int start, int T, int nblk, long long C) {
  long long cost = 0;
  int it = start;
  while (it < T) {
    const int k0 = it % nblk, room = nblk - k0;
    const long long rest_of_unit = 2LL * room + (k0 ? kPieceCostPartial : kPieceCostWhole);
    if (cost + rest_of_unit <= C) {
      cost += rest_of_unit;
      it += room;
      continue;
    }
    const long long cnt = (C - cost - kPieceCostPartial) / 2;  // a partial piece that ends inside the unit
    if (cnt >= 1) it += (int)(cnt < room - 1 ? cnt : room - 1);
    break;
  }
  return it;
}

// Spans of cost at most C, left to right; the number of spans, or 0 when C is too small for some span or more
// than `gmax` spans would be needed.
int cut_spans(int T, int nblk, long long C, int gmax, int* bounds) {
  int g = 0, it = 0;
  bounds[0] = 0;
  while (it < T) {
    if (g == gmax) return 0;
    const int end = span_end(it, T, nblk, C);
    if (end == it) return 0;
    bounds[++g] = it = end;
  }
  return g;
}

// Whole units per CTA when that is at most kSplitCostTiles tiles slower than a perfectly even cut;
// otherwise spans cut at single key tiles: evenly where a span holds two units or more (the pieces' costs are
// small beside it), else so that the longest span, pieces' costs included, is as short as possible (the
// smallest budget C for which a left-to-right cut needs no more spans than there are CTAs).
Spans plan_spans(int units, int nblk) {
  Spans sp = {};
  sp.nblk = nblk;
  sp.T = units * nblk;
  const int gmax = max_ctas();
  const int whole_tiles = ((units + gmax - 1) / gmax) * nblk;  // longest CTA with whole units
  const int even_tiles = (sp.T + gmax - 1) / gmax;             // longest CTA with an even cut
  int mode = whole_tiles <= even_tiles + kSplitCostTiles ? 0 : 1;
  const int forced = g_tune_attention_split.load(std::memory_order_relaxed);  // test-only override
  if (forced == 0 || forced == 1) mode = forced;
  sp.split = mode;
  const int quantum = mode == 0 ? nblk : 1;
  const int quanta = sp.T / quantum;
  sp.G = quanta < gmax ? quanta : gmax;
  const int q = quanta / sp.G, r = quanta - q * sp.G;  // the first r spans hold q + 1 quanta, the others q
  for (int g = 0; g <= sp.G; ++g) sp.bounds[g] = (g * q + (g < r ? g : r)) * quantum;
  if (mode == 1 && q >= 2 * nblk) {
    // long spans: the even cut, with every bound that falls within kSnapTiles of a unit boundary moved onto it
    for (int g = 1; g < sp.G; ++g) {
      const int unit_edge = (sp.bounds[g] + nblk / 2) / nblk * nblk;
      const int off = sp.bounds[g] - unit_edge;
      if (off != 0 && off >= -kSnapTiles && off <= kSnapTiles) sp.bounds[g] = unit_edge;
    }
  } else if (mode == 1) {
    // spans of less than two units: the pieces' costs decide
    long long lo = 2 + kPieceCostPartial, hi = 2LL * sp.T + (long long)kPieceCostPartial * (units + 2);
    while (lo < hi) {  // cut_spans succeeds for every budget from some value on
      const long long mid = (lo + hi) / 2;
      if (cut_spans(sp.T, nblk, mid, gmax, sp.bounds)) hi = mid;
      else lo = mid + 1;
    }
    sp.G = cut_spans(sp.T, nblk, lo, gmax, sp.bounds);
  }
  for (int g = 0; g < sp.G; ++g) {
    const int unit[2] = {sp.bounds[g] / nblk, (sp.bounds[g + 1] - 1) / nblk};
    for (int e = 0; e < 2; ++e) {
      sp.unit_lo[e][g] = (uint8_t)sp.owner(unit[e] * nblk);
      sp.unit_hi[e][g] = (uint8_t)sp.owner((unit[e] + 1) * nblk - 1);
    }
  }
  return sp;
}

template <int DH>
cudaError_t launch(int B, int L, int heads, const void* q, const void* k, const void* v, void* o, void* ws,
                   bool tickets_clean, uint32_t* dev_status, cudaStream_t s) {
  using C = AttCfg<DH>;
  CUtensorMap tq, tk, tv, to;
  const uint64_t dims[3] = {(uint64_t)heads * DH, (uint64_t)L, (uint64_t)B};
  const uint64_t strides[2] = {(uint64_t)heads * DH * 2, (uint64_t)L * heads * DH * 2};
  const uint32_t box_q[3] = {64, kBM, 1};
  const uint32_t box_kv[3] = {64, kBN, 1};
  const uint32_t box_o[3] = {64, 32, 1};  // a softmax warp's 32 rows of one 64-channel slab
  if (!encode_tmap_16bit(&tq, q, 3, dims, strides, box_q) || !encode_tmap_16bit(&tk, k, 3, dims, strides, box_kv) ||
      !encode_tmap_16bit(&tv, v, 3, dims, strides, box_kv) || !encode_tmap_16bit(&to, o, 3, dims, strides, box_o))
    return cudaErrorInvalidValue;
  static std::atomic<unsigned long long> smem_raised{0};
  cudaError_t e = raise_dynamic_smem(attention_tc_kernel<DH>, C::kSmemBytes, smem_raised);
  if (e != cudaSuccess) return e;
  const long long units = (long long)B * heads * ((L + kUM - 1) / kUM);
  const int nblk = (L + kBN - 1) / kBN;
  if (units * nblk > 0x7fffffffLL) return cudaErrorInvalidValue;  // iteration indices are 32-bit
  const Spans sp = plan_spans((int)units, nblk);
  const size_t tb = ticket_bytes(B, L, heads);
  if (sp.split && !tickets_clean) {  // units are split: their tickets start at zero
    e = cudaMemsetAsync(ws, 0, tb, s);
    if (e != cudaSuccess) return e;
  }
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  e = launch_dependent(attention_tc_kernel<DH>, dim3(sp.G), dim3(kThreads), (size_t)C::kSmemBytes, s, tq, tk, tv, to,
                       (__nv_bfloat16*)o, L, heads, scale_log2, sp, (uint32_t*)ws, (float*)((char*)ws + tb), dev_status);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace

size_t attention_tc_workspace_bytes(int B, int L, int heads, int dh) {
  const size_t piece = (dh == 64 ? piece_floats<64>() : piece_floats<128>()) * sizeof(float);
  return ticket_bytes(B, L, heads) + 2 * (size_t)kMaxCtas * piece;
}

size_t attention_tc_ticket_bytes(int B, int L, int heads) { return ticket_bytes(B, L, heads); }

int attention_tc_plan(int B, int L, int heads, int info[4], int* bounds, int* owner_first, int* owner_last, int capacity) {
  const long long units = (long long)B * heads * ((L + kUM - 1) / kUM);
  const int nblk = (L + kBN - 1) / kBN;
  if (units * nblk > 0x7fffffffLL) return 0;
  const Spans sp = plan_spans((int)units, nblk);
  info[0] = sp.G;
  info[1] = sp.split;
  info[2] = (int)units;
  info[3] = nblk;
  for (int g = 0; g <= sp.G && g < capacity; ++g) {
    if (bounds) bounds[g] = sp.bound(g);
    if (g < sp.G && sp.split) {
      if (owner_first) owner_first[g] = sp.owner(sp.bound(g));
      if (owner_last) owner_last[g] = sp.owner(sp.bound(g + 1) - 1);
    }
  }
  return sp.G;
}

cudaError_t launch_attention_tc(int B, int L, int heads, int dh, const void* q, const void* k, const void* v, void* o,
                                void* ws, bool tickets_clean, uint32_t* dev_status, cudaStream_t s) {
  if (dh == 64) return launch<64>(B, L, heads, q, k, v, o, ws, tickets_clean, dev_status, s);
  if (dh == 128) return launch<128>(B, L, heads, q, k, v, o, ws, tickets_clean, dev_status, s);
  return cudaErrorInvalidValue;
}

}  // namespace toma
