// extern "C" boundary of the ToMA library: descriptor validation, workspace
// carve-up and kernel sequencing.  Argument marshalling only; all arithmetic is in
// the kernels.
#include <math.h>

#include "common.cuh"

namespace toma {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

toma_status make_geom(const toma_desc* desc, Geom* g) {
  if (!desc) return TOMA_ERR_NULL;
  if (desc->dtype != TOMA_BF16 && desc->dtype != TOMA_F32) return TOMA_ERR_DTYPE;
  if (desc->batch < 1 || desc->grid_h < 1 || desc->grid_w < 1 || desc->dim < 8 || desc->dim % 8) return TOMA_ERR_SHAPE;
  if (desc->tile_h < 1 || desc->tile_w < 1 || desc->grid_h % desc->tile_h || desc->grid_w % desc->tile_w)
    return TOMA_ERR_SHAPE;
  if (desc->n_extra < 0) return TOMA_ERR_SHAPE;
  if (desc->n_heads < 1 || desc->head_dim < 1 || (long long)desc->n_heads * desc->head_dim != desc->dim)
    return TOMA_ERR_SHAPE;
  if (!(desc->merge_ratio >= 0.f) || !(desc->merge_ratio < 1.f)) return TOMA_ERR_RATIO;
  if (!(desc->tau > 0.f) || !isfinite(desc->tau)) return TOMA_ERR_TAU;
  if (desc->reuse_interval < 1 || desc->weight_reuse_interval < 0) return TOMA_ERR_SHAPE;
  const long long nloc = (long long)desc->tile_h * desc->tile_w;
  if (nloc > kMaxNloc || desc->dim > kMaxDim) return TOMA_ERR_UNSUPPORTED;
  const long long ntok = (long long)desc->grid_h * desc->grid_w;
  if ((ntok + desc->n_extra) * (long long)desc->batch > (1ll << 30)) return TOMA_ERR_UNSUPPORTED;
  const int dloc = (int)nloc - (int)lround((double)desc->merge_ratio * (double)nloc);
  if (dloc < 1 || dloc > nloc) return TOMA_ERR_RATIO;
  g->B = desc->batch; g->H = desc->grid_h; g->W = desc->grid_w; g->d = desc->dim;
  g->th = desc->tile_h; g->tw = desc->tile_w;
  g->tiles_x = desc->grid_w / desc->tile_w;
  g->P = g->tiles_x * (desc->grid_h / desc->tile_h);
  g->N = (int)ntok; g->Nloc = (int)nloc; g->Dloc = dloc; g->D = g->P * dloc;
  g->n_extra = desc->n_extra; g->Lm = g->D + g->n_extra;
  g->heads = desc->n_heads; g->dh = desc->head_dim;
  g->f32 = desc->dtype == TOMA_F32;
  if (desc->global_merge != 0 && desc->global_merge != 1) return TOMA_ERR_SHAPE;
  g->global_merge = desc->global_merge == 1;
  if (g->global_merge && (long long)g->N * g->D > (1ll << 27)) return TOMA_ERR_UNSUPPORTED;  // dense D x N weights per image
  if (desc->unmerge_mode != TOMA_UNMERGE_TRANSPOSE && desc->unmerge_mode != TOMA_UNMERGE_SHARES) return TOMA_ERR_SHAPE;
  g->unmerge_mode = desc->unmerge_mode;
  g->logit_scale = (float)(1.0 / ((double)desc->tau * sqrt((double)desc->dim)));
  return TOMA_OK;
}

static bool attention_on_tc(int dh, bool f32) { return !f32 && (dh == 64 || dh == 128); }

static size_t attention_ws_bytes(int B, int L, int heads, int dh, bool f32) {
  return attention_on_tc(dh, f32) ? attention_tc_workspace_bytes(B, L, heads, dh) : 0;
}

// Bytes of one matrix of the weight buffer (one fp32 plane, or a hi and a lo bf16 plane, per region).
static size_t weight_matrix_bytes(const Geom& g) {
  const Geom gm = merge_geom(g);
  return (size_t)gm.B * gm.P * gm.Nloc * gm.Dloc * 4;
}
// The matrix toma_unmerge reads.
static const void* unmerge_matrix(const Geom& g, const void* w) {
  return g.unmerge_mode == TOMA_UNMERGE_TRANSPOSE ? w : (const char*)w + weight_matrix_bytes(g);
}

Geom merge_geom(const Geom& g) {
  Geom m = g;
  if (g.global_merge) {
    m.P = 1; m.tiles_x = 1; m.th = g.H; m.tw = g.W; m.Nloc = g.N; m.Dloc = g.D;
  }
  return m;
}

WsLayout ws_layout(const Geom& g) {
  WsLayout l;
  const Geom gm = merge_geom(g);
  const size_t tiles = (size_t)g.B * g.P;
  const size_t esz = g.f32 ? 4 : 2;
  size_t off = 0;
  l.y_off = off;      off = align_up(off + tiles * g.Nloc * g.d * sizeof(__nv_bfloat16), 256);
  l.sq_off = off;     off = align_up(off + tiles * g.Nloc * g.Nloc * sizeof(int16_t), 256);
  l.logits_off = off; off = align_up(off + (size_t)gm.B * gm.P * gm.Dloc * gm.Nloc * sizeof(float), 256);
  l.wts_off = off;    off = align_up(off + (weights_tc_supported(gm) ? weights_tc_scratch_bytes(gm) : 0), 256);
  l.gidx_off = off;   off = align_up(off + (g.global_merge ? (size_t)g.B * g.D * sizeof(int32_t) : 0), 256);
  l.xm_off = off;     off = align_up(off + (size_t)g.B * g.Lm * g.d * esz, 256);
  l.att_off = off;    off = align_up(off + (size_t)g.B * g.Lm * g.d * esz, 256);
  l.att_ws_off = off; off = align_up(off + attention_ws_bytes(g.B, g.Lm, g.heads, g.dh, g.f32), 256);
  // q, k, v and the projected attention output of toma_block_proj (four merged-size tensors)
  l.proj_off = off;   off = align_up(off + 4 * align_up((size_t)g.B * g.Lm * g.d * esz, 256), 256);
  l.total = off;
  return l;
}

static bool attention_supported_simt(int dh) { return dh == 16 || dh == 32 || dh == 64 || dh == 128; }

static toma_status check_ws(const Geom& g, const void* ws, size_t ws_bytes) {
  if (!ws) return TOMA_ERR_WORKSPACE;
  if (((uintptr_t)ws & 15) != 0) return TOMA_ERR_WORKSPACE;
  return ws_bytes >= ws_layout(g).total ? TOMA_OK : TOMA_ERR_WORKSPACE;
}

static toma_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? TOMA_OK : TOMA_ERR_CUDA; }

static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

// --- step sequencing shared by the public entry points -------------------------------

static cudaError_t do_select(const Geom& g, const void* x, int32_t* idx, char* ws, uint32_t* dev_status,
                             cudaStream_t s) {
  const WsLayout l = ws_layout(g);
  __nv_bfloat16* y = (__nv_bfloat16*)(ws + l.y_off);
  int16_t* sq = (int16_t*)(ws + l.sq_off);
  cudaError_t e = launch_quantise(g, x, y, s);
  if (e != cudaSuccess) return e;
  e = gram_tc_supported(g) ? launch_gram_tc(g, y, sq, dev_status, s) : launch_gram_ffma(g, y, sq, s);
  if (e != cudaSuccess) return e;
  return launch_greedy(g, sq, idx, s);
}

static cudaError_t do_weights(const Geom& g, const void* x, const int32_t* idx, void* w, char* ws,
                              uint32_t* dev_status, cudaStream_t s) {
  const WsLayout l = ws_layout(g);
  const Geom gm = merge_geom(g);
  if (g.global_merge) {  // image-level destination ids; from here on the image is one region
    int32_t* gidx = (int32_t*)(ws + l.gidx_off);
    cudaError_t e = launch_global_idx(g, idx, gidx, s);
    if (e != cudaSuccess) return e;
    idx = gidx;
  }
  void* wu = g.unmerge_mode == TOMA_UNMERGE_SHARES ? (char*)w + weight_matrix_bytes(g) : nullptr;
  if (weights_tc_supported(gm))
    return launch_weights_tc(gm, x, idx, w, wu, (float*)(ws + l.logits_off), ws + l.wts_off, dev_status, s);
  return launch_weights_simt(gm, x, idx, w, wu, (float*)(ws + l.logits_off), s);
}

// `zero`, `zero_bytes`: a region to clear on the side; *zeroed says whether the path taken did it.
static cudaError_t do_merge(const Geom& g_sel, const void* w, const void* x, void* xm, void* zero, size_t zero_bytes,
                            bool* zeroed, uint32_t* dev_status, cudaStream_t s) {
  if (zeroed) *zeroed = false;
  const Geom g = merge_geom(g_sel);
  if (linear_tc_supported(g)) {
    cudaError_t e = launch_merge_tc(g, w, x, xm, zero, zero_bytes, dev_status, s);
    if (zeroed) *zeroed = e == cudaSuccess && zero_bytes > 0;
    return e != cudaSuccess ? e : launch_copy_extra(g, x, xm, true, s);
  }
  return launch_merge_simt(g, w, x, xm, s);
}

static cudaError_t do_unmerge(const Geom& g_sel, const void* w, const void* y, void* out, uint32_t* dev_status,
                              cudaStream_t s) {
  const Geom g = merge_geom(g_sel);
  w = unmerge_matrix(g_sel, w);
  if (linear_tc_supported(g)) {
    cudaError_t e = launch_unmerge_tc(g, w, y, out, dev_status, s);
    return e != cudaSuccess ? e : launch_copy_extra(g, y, out, false, s);
  }
  return launch_unmerge_simt(g, w, y, out, s);
}

static cudaError_t do_attention(int B, int L, int heads, int dh, bool f32, const void* q, const void* k,
                                const void* v, void* o, void* att_ws, bool tickets_clean, uint32_t* dev_status,
                                cudaStream_t s) {
  if (attention_on_tc(dh, f32))
    return launch_attention_tc(B, L, heads, dh, q, k, v, o, att_ws, tickets_clean, dev_status, s);
  return launch_attention_simt(B, L, heads, dh, f32, q, k, v, o, s);
}

}  // namespace toma

using namespace toma;

extern "C" {

toma_status toma_validate(const toma_desc* desc) {
  Geom g;
  return make_geom(desc, &g);
}

size_t toma_workspace_bytes(const toma_desc* desc) {
  Geom g;
  if (make_geom(desc, &g) != TOMA_OK) return 0;
  return ws_layout(g).total;
}

size_t toma_weights_bytes(const toma_desc* desc) {
  Geom g;
  if (make_geom(desc, &g) != TOMA_OK) return 0;
  return weight_matrix_bytes(g) * (g.unmerge_mode == TOMA_UNMERGE_TRANSPOSE ? 1 : 2);
}

int32_t toma_dest_per_tile(const toma_desc* desc) {
  Geom g;
  if (make_geom(desc, &g) != TOMA_OK) return -1;
  return g.Dloc;
}

const char* toma_status_str(toma_status s) {
  switch (s) {
    case TOMA_OK: return "ok";
    case TOMA_ERR_NULL: return "null pointer";
    case TOMA_ERR_SHAPE: return "bad shape";
    case TOMA_ERR_DTYPE: return "bad dtype";
    case TOMA_ERR_RATIO: return "bad merge ratio";
    case TOMA_ERR_TAU: return "bad temperature";
    case TOMA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TOMA_ERR_UNSUPPORTED: return "unsupported size";
    case TOMA_ERR_CUDA: return "CUDA error";
    case TOMA_ERR_TIMEOUT: return "device-side wait timed out";
    case TOMA_ERR_SCRATCH_LIMIT: return "problem does not fit the built-in static scratch";
  }
  return "unknown";
}

toma_status toma_select(const toma_desc* desc, const void* x, int32_t* idx, void* ws, size_t ws_bytes,
                        uint32_t* dev_status, void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!x || !idx) return TOMA_ERR_NULL;
  if (misaligned(x)) return TOMA_ERR_SHAPE;
  if ((st = check_ws(g, ws, ws_bytes)) != TOMA_OK) return st;
  return cuda_ok(do_select(g, x, idx, (char*)ws, dev_status, (cudaStream_t)stream));
}

toma_status toma_merge_weights(const toma_desc* desc, const void* x, const int32_t* idx, void* w, void* ws,
                               size_t ws_bytes, uint32_t* dev_status, void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!x || !idx || !w) return TOMA_ERR_NULL;
  if (misaligned(x) || misaligned(w)) return TOMA_ERR_SHAPE;
  if ((st = check_ws(g, ws, ws_bytes)) != TOMA_OK) return st;
  return cuda_ok(do_weights(g, x, idx, w, (char*)ws, dev_status, (cudaStream_t)stream));
}

toma_status toma_merge(const toma_desc* desc, const void* w, const void* x, void* xm, uint32_t* dev_status,
                       void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!w || !x || !xm) return TOMA_ERR_NULL;
  if (misaligned(x) || misaligned(w) || misaligned(xm)) return TOMA_ERR_SHAPE;
  return cuda_ok(do_merge(g, w, x, xm, nullptr, 0, nullptr, dev_status, (cudaStream_t)stream));
}

toma_status toma_unmerge(const toma_desc* desc, const void* w, const void* y, void* out, uint32_t* dev_status,
                         void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!w || !y || !out) return TOMA_ERR_NULL;
  if (misaligned(y) || misaligned(w) || misaligned(out)) return TOMA_ERR_SHAPE;
  return cuda_ok(do_unmerge(g, w, y, out, dev_status, (cudaStream_t)stream));
}

size_t toma_attention_workspace_bytes(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype) {
  if ((dtype != TOMA_BF16 && dtype != TOMA_F32) || batch < 1 || len < 1 || n_heads < 1 || head_dim < 1) return 0;
  return attention_ws_bytes(batch, len, n_heads, head_dim, dtype == TOMA_F32);
}

int32_t toma_attention_plan(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype, int32_t info[4],
                            int32_t* bounds, int32_t* owner_first, int32_t* owner_last, int32_t capacity) {
  if (!info || batch < 1 || len < 1 || n_heads < 1 || !attention_on_tc(head_dim, dtype == TOMA_F32)) return 0;
  return attention_tc_plan(batch, len, n_heads, info, bounds, owner_first, owner_last, capacity);
}

toma_status toma_attention(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype,
                           const void* q, const void* k, const void* v, void* o, void* ws, size_t ws_bytes,
                           uint32_t* dev_status, void* stream) {
  if (dtype != TOMA_BF16 && dtype != TOMA_F32) return TOMA_ERR_DTYPE;
  if (batch < 1 || len < 1 || n_heads < 1 || head_dim < 1) return TOMA_ERR_SHAPE;
  if (!q || !k || !v || !o) return TOMA_ERR_NULL;
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(o)) return TOMA_ERR_SHAPE;
  if (!attention_supported_simt(head_dim)) return TOMA_ERR_UNSUPPORTED;
  const size_t need = attention_ws_bytes(batch, len, n_heads, head_dim, dtype == TOMA_F32);
  if (need > 0 && (!ws || misaligned(ws) || ws_bytes < need)) return TOMA_ERR_WORKSPACE;
  return cuda_ok(do_attention(batch, len, n_heads, head_dim, dtype == TOMA_F32, q, k, v, o, ws, false, dev_status,
                              (cudaStream_t)stream));
}

// c[i] = a w[i] for n_mats weight / output pairs
static cudaError_t do_linear(int M, int N, int K, bool f32, const void* a, const void* const* w, void* const* c, int n_mats,
                             int act, uint32_t* dev_status, cudaStream_t s) {
  if (!f32 && linear_tc_shape_ok(M, N, K)) return launch_linear_tc(M, N, K, a, w, c, n_mats, act, dev_status, s);
  for (int i = 0; i < n_mats; ++i) {
    cudaError_t e = launch_linear_simt(M, N, K, f32, a, w[i], c[i], act, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

toma_status toma_linear(int32_t m, int32_t n, int32_t k, int32_t dtype, const void* a, const void* w, void* c,
                        uint32_t* dev_status, void* stream) {
  if (dtype != TOMA_BF16 && dtype != TOMA_F32) return TOMA_ERR_DTYPE;
  if (m < 1 || n < 1 || k < 1) return TOMA_ERR_SHAPE;
  if (!a || !w || !c) return TOMA_ERR_NULL;
  if (misaligned(a) || misaligned(w) || misaligned(c)) return TOMA_ERR_SHAPE;
  if (dtype == TOMA_BF16 && (n % 8 || k % 8)) return TOMA_ERR_SHAPE;  // 16-byte rows
  const void* ws[1] = {w};
  void* cs[1] = {c};
  return cuda_ok(do_linear(m, n, k, dtype == TOMA_F32, a, ws, cs, 1, kActNone, dev_status, (cudaStream_t)stream));
}

// Every host-detectable error of a block call, checked before anything is enqueued.
static toma_status block_check(const toma_desc* desc, int32_t step, const void* x, const void* const* proj,
                               const void* const* mlp, int hidden, const void* out, const int32_t* idx_state,
                               const void* w_state, const void* ws, size_t ws_bytes, Geom* geom) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!x || !out || !idx_state || !w_state) return TOMA_ERR_NULL;
  if (proj)
    for (int i = 0; i < 4; ++i) {
      if (!proj[i]) return TOMA_ERR_NULL;
      if (misaligned(proj[i])) return TOMA_ERR_SHAPE;
    }
  if (mlp) {
    if (!mlp[0] || !mlp[1]) return TOMA_ERR_NULL;
    if (misaligned(mlp[0]) || misaligned(mlp[1])) return TOMA_ERR_SHAPE;
    // the hidden tensor lives in the four merged-size slots of the projection scratch
    if (hidden < 8 || hidden % 8 || hidden > 4 * g.d) return TOMA_ERR_SHAPE;
  }
  if (step < 0) return TOMA_ERR_SHAPE;
  if (misaligned(x) || misaligned(out) || misaligned(w_state)) return TOMA_ERR_SHAPE;
  if (!attention_supported_simt(g.dh)) return TOMA_ERR_UNSUPPORTED;
  if ((st = check_ws(g, ws, ws_bytes)) != TOMA_OK) return st;
  *geom = g;
  return TOMA_OK;
}

// The wrapped module F: attention over the merged tokens with Q = K = V = X_m, or, with projection weights
// (proj = {wq, wk, wv, wo}, each [dim][dim], row-major [in][out]), the whole attention module
// (X_m wq, X_m wk, X_m wv -> attention -> wo); or, with mlp = {w1 [dim][hidden], w2 [hidden][dim]}, the MLP
// GELU(X_m w1) w2.
static toma_status block_impl(const toma_desc* desc, int32_t step, const void* x, const void* const* proj,
                              const void* const* mlp, int hidden, void* out, int32_t* idx_state, void* w_state, void* ws,
                              size_t ws_bytes, uint32_t* dev_status, void* stream) {
  Geom g;
  toma_status st = block_check(desc, step, x, proj, mlp, hidden, out, idx_state, w_state, ws, ws_bytes, &g);
  if (st != TOMA_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  const WsLayout l = ws_layout(g);
  const int kw = desc->weight_reuse_interval > 0 ? desc->weight_reuse_interval : desc->reuse_interval;
  const bool refresh_sel = step % desc->reuse_interval == 0;
  const bool refresh_w = refresh_sel || step % kw == 0;
  cudaError_t e = cudaSuccess;
  const bool unfused = g_tune_block_unfused.load(std::memory_order_relaxed) != 0;
  if (refresh_sel && refresh_w && refresh_fused_supported(g) && !unfused) {
    // small tiles: Gram, greedy rounds and weights of a tile in one kernel behind the quantisation
    __nv_bfloat16* y = (__nv_bfloat16*)(wsb + l.y_off);
    e = launch_quantise(g, x, y, s);
    if (e == cudaSuccess) e = launch_refresh_fused(g, y, x, idx_state, w_state, dev_status, s);
  } else if (refresh_sel && refresh_w && weights_gram_supported(g) && !unfused) {
    // few large tiles: the raw Gram matrix of every tile is computed on the SMs that idle during the greedy rounds
    // (it takes the place of the quantised tokens, dead by then), and the weights are read out of it
    float* G = (float*)(wsb + l.y_off);
    e = do_select(g, x, idx_state, wsb, dev_status, s);
    if (e == cudaSuccess) e = launch_gram_raw(g, x, G, dev_status, s);
    if (e == cudaSuccess) e = launch_weights_gram(g, G, idx_state, w_state, dev_status, s);
  } else {
    if (refresh_sel) e = do_select(g, x, idx_state, wsb, dev_status, s);
    if (e == cudaSuccess && refresh_w) e = do_weights(g, x, idx_state, w_state, wsb, dev_status, s);
  }
  // merge, attention and unmerge as one kernel where the shape allows (small tiles, few merged tokens)
  if (!proj && !mlp && block_fused_supported(g) && !unfused && block_fused_launchable(g)) {
    if (e == cudaSuccess) e = launch_block_fused(g, w_state, x, out, dev_status, s);
    return cuda_ok(e);
  }
  void* xm = wsb + l.xm_off;
  void* att = wsb + l.att_off;
  // the merge kernel clears the attention kernel's tickets on the side (saves a memset between them)
  bool tickets_clean = false;
  const size_t ticket_bytes = attention_on_tc(g.dh, g.f32) ? attention_tc_ticket_bytes(g.B, g.Lm, g.heads) : 0;
  if (e == cudaSuccess) e = do_merge(g, w_state, x, xm, wsb + l.att_ws_off, ticket_bytes, &tickets_clean, dev_status, s);
  if (mlp) {
    const int rows = g.B * g.Lm;
    void* hid[1] = {wsb + l.proj_off};
    void* ys[1] = {att};
    if (e == cudaSuccess) e = do_linear(rows, hidden, g.d, g.f32, xm, mlp, hid, 1, kActGelu, dev_status, s);
    if (e == cudaSuccess) e = do_linear(rows, g.d, hidden, g.f32, hid[0], mlp + 1, ys, 1, kActNone, dev_status, s);
    if (e == cudaSuccess) e = do_unmerge(g, w_state, att, out, dev_status, s);
    return cuda_ok(e);
  }
  if (!proj) {
    if (e == cudaSuccess) e = do_attention(g.B, g.Lm, g.heads, g.dh, g.f32, xm, xm, xm, att, wsb + l.att_ws_off, tickets_clean, dev_status, s);
    if (e == cudaSuccess) e = do_unmerge(g, w_state, att, out, dev_status, s);
    return cuda_ok(e);
  }
  const size_t one = align_up((size_t)g.B * g.Lm * g.d * (g.f32 ? 4 : 2), 256);
  void* qkv[3] = {wsb + l.proj_off, wsb + l.proj_off + one, wsb + l.proj_off + 2 * one};
  void* y = wsb + l.proj_off + 3 * one;
  const int rows = g.B * g.Lm;
  if (e == cudaSuccess) e = do_linear(rows, g.d, g.d, g.f32, xm, proj, qkv, 3, kActNone, dev_status, s);
  if (e == cudaSuccess) e = do_attention(g.B, g.Lm, g.heads, g.dh, g.f32, qkv[0], qkv[1], qkv[2], att, wsb + l.att_ws_off, tickets_clean, dev_status, s);
  void* ys[1] = {y};
  if (e == cudaSuccess) e = do_linear(rows, g.d, g.d, g.f32, att, proj + 3, ys, 1, kActNone, dev_status, s);
  if (e == cudaSuccess) e = do_unmerge(g, w_state, y, out, dev_status, s);
  return cuda_ok(e);
}

toma_status toma_block(const toma_desc* desc, int32_t step, const void* x, void* out, int32_t* idx_state,
                       void* w_state, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream) {
  return block_impl(desc, step, x, nullptr, nullptr, 0, out, idx_state, w_state, ws, ws_bytes, dev_status, stream);
}

toma_status toma_block_mlp(const toma_desc* desc, int32_t step, const void* x, const void* w1, const void* w2,
                           int32_t hidden, void* out, int32_t* idx_state, void* w_state, void* ws, size_t ws_bytes,
                           uint32_t* dev_status, void* stream) {
  const void* mlp[2] = {w1, w2};
  return block_impl(desc, step, x, nullptr, mlp, hidden, out, idx_state, w_state, ws, ws_bytes, dev_status, stream);
}

size_t toma_mlp_workspace_bytes(int32_t rows, int32_t dim, int32_t hidden, int32_t dtype) {
  if ((dtype != TOMA_BF16 && dtype != TOMA_F32) || rows < 1 || dim < 1 || hidden < 1) return 0;
  return align_up((size_t)rows * hidden * (dtype == TOMA_F32 ? 4 : 2), 256);
}

toma_status toma_mlp(int32_t rows, int32_t dim, int32_t hidden, int32_t dtype, const void* x, const void* w1, const void* w2,
                     void* out, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream) {
  if (dtype != TOMA_BF16 && dtype != TOMA_F32) return TOMA_ERR_DTYPE;
  if (rows < 1 || dim < 1 || hidden < 1) return TOMA_ERR_SHAPE;
  if (!x || !w1 || !w2 || !out) return TOMA_ERR_NULL;
  if (misaligned(x) || misaligned(w1) || misaligned(w2) || misaligned(out)) return TOMA_ERR_SHAPE;
  if (dtype == TOMA_BF16 && (dim % 8 || hidden % 8)) return TOMA_ERR_SHAPE;  // 16-byte rows
  if (!ws || misaligned(ws) || ws_bytes < toma_mlp_workspace_bytes(rows, dim, hidden, dtype)) return TOMA_ERR_WORKSPACE;
  const bool f32 = dtype == TOMA_F32;
  cudaStream_t s = (cudaStream_t)stream;
  const void* w1s[1] = {w1};
  const void* w2s[1] = {w2};
  void* hid[1] = {ws};
  void* outs[1] = {out};
  cudaError_t e = do_linear(rows, hidden, dim, f32, x, w1s, hid, 1, kActGelu, dev_status, s);
  if (e == cudaSuccess) e = do_linear(rows, dim, hidden, f32, ws, w2s, outs, 1, kActNone, dev_status, s);
  return cuda_ok(e);
}

toma_status toma_block_proj(const toma_desc* desc, int32_t step, const void* x, const void* wq, const void* wk,
                            const void* wv, const void* wo, void* out, int32_t* idx_state, void* w_state, void* ws,
                            size_t ws_bytes, uint32_t* dev_status, void* stream) {
  const void* proj[4] = {wq, wk, wv, wo};
  return block_impl(desc, step, x, proj, nullptr, 0, out, idx_state, w_state, ws, ws_bytes, dev_status, stream);
}

size_t toma_attention_proj_workspace_bytes(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype) {
  if ((dtype != TOMA_BF16 && dtype != TOMA_F32) || batch < 1 || len < 1 || n_heads < 1 || head_dim < 1) return 0;
  const size_t one = align_up((size_t)batch * len * n_heads * head_dim * (dtype == TOMA_F32 ? 4 : 2), 256);
  return 4 * one + align_up(attention_ws_bytes(batch, len, n_heads, head_dim, dtype == TOMA_F32), 256);
}

toma_status toma_attention_proj(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype, const void* x,
                                const void* wq, const void* wk, const void* wv, const void* wo, void* out, void* ws,
                                size_t ws_bytes, uint32_t* dev_status, void* stream) {
  if (dtype != TOMA_BF16 && dtype != TOMA_F32) return TOMA_ERR_DTYPE;
  if (batch < 1 || len < 1 || n_heads < 1 || head_dim < 1) return TOMA_ERR_SHAPE;
  if (!x || !wq || !wk || !wv || !wo || !out) return TOMA_ERR_NULL;
  if (misaligned(x) || misaligned(wq) || misaligned(wk) || misaligned(wv) || misaligned(wo) || misaligned(out)) return TOMA_ERR_SHAPE;
  if (!attention_supported_simt(head_dim)) return TOMA_ERR_UNSUPPORTED;
  const bool f32 = dtype == TOMA_F32;
  const int d = n_heads * head_dim;
  if (d % 8) return TOMA_ERR_SHAPE;
  if (!ws || misaligned(ws) || ws_bytes < toma_attention_proj_workspace_bytes(batch, len, n_heads, head_dim, dtype)) return TOMA_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  const size_t one = align_up((size_t)batch * len * d * (f32 ? 4 : 2), 256);
  void* qkv[3] = {wsb, wsb + one, wsb + 2 * one};
  void* att = wsb + 3 * one;
  void* att_ws = wsb + 4 * one;
  const void* proj[4] = {wq, wk, wv, wo};
  const int rows = batch * len;
  cudaError_t e = do_linear(rows, d, d, f32, x, proj, qkv, 3, kActNone, dev_status, s);
  if (e == cudaSuccess) e = do_attention(batch, len, n_heads, head_dim, f32, qkv[0], qkv[1], qkv[2], att, att_ws, false, dev_status, s);
  void* outs[1] = {out};
  if (e == cudaSuccess) e = do_linear(rows, d, d, f32, att, proj + 3, outs, 1, kActNone, dev_status, s);
  return cuda_ok(e);
}

toma_status toma_block_host(const toma_desc* desc, int32_t step, const void* x_host, void* out_host, void* x_dev,
                            void* out_dev, int32_t* idx_state, void* w_state, void* ws, size_t ws_bytes,
                            uint32_t* dev_status, void* stream, void* copy_in_stream, void* copy_out_stream,
                            void* copied_in_event, void* computed_event) {
  if (!x_host || !out_host) return TOMA_ERR_NULL;
  Geom g;  // the same checks toma_block makes, before the first copy is enqueued
  toma_status st = block_check(desc, step, x_dev, nullptr, nullptr, 0, out_dev, idx_state, w_state, ws, ws_bytes, &g);
  if (st != TOMA_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  cudaStream_t s_in = copy_in_stream ? (cudaStream_t)copy_in_stream : s;
  cudaStream_t s_out = copy_out_stream ? (cudaStream_t)copy_out_stream : s;
  if ((s_in != s && !copied_in_event) || (s_out != s && !computed_event)) return TOMA_ERR_NULL;
  const size_t bytes = (size_t)g.B * (size_t)g.tokens_all() * g.d * (g.f32 ? 4 : 2);
  if (cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, s_in) != cudaSuccess) return TOMA_ERR_CUDA;
  if (s_in != s) {
    if (cudaEventRecord((cudaEvent_t)copied_in_event, s_in) != cudaSuccess) return TOMA_ERR_CUDA;
    if (cudaStreamWaitEvent(s, (cudaEvent_t)copied_in_event, 0) != cudaSuccess) return TOMA_ERR_CUDA;
  }
  st = toma_block(desc, step, x_dev, out_dev, idx_state, w_state, ws, ws_bytes, dev_status, stream);
  if (st != TOMA_OK) return st;
  if (s_out != s) {
    if (cudaEventRecord((cudaEvent_t)computed_event, s) != cudaSuccess) return TOMA_ERR_CUDA;
    if (cudaStreamWaitEvent(s_out, (cudaEvent_t)computed_event, 0) != cudaSuccess) return TOMA_ERR_CUDA;
  }
  return cuda_ok(cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, s_out));
}

toma_status toma_weights_export(const toma_desc* desc, const void* w, float* dense, void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!w || !dense) return TOMA_ERR_NULL;
  return cuda_ok(launch_weights_export(merge_geom(g), w, dense, (cudaStream_t)stream));
}

toma_status toma_weights_import(const toma_desc* desc, const float* dense, void* w, void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!w || !dense) return TOMA_ERR_NULL;
  cudaError_t e = launch_weights_import(merge_geom(g), dense, w, (cudaStream_t)stream);
  if (e == cudaSuccess && g.unmerge_mode != TOMA_UNMERGE_TRANSPOSE)
    e = launch_weights_import(merge_geom(g), dense, (char*)w + weight_matrix_bytes(g), (cudaStream_t)stream);
  return cuda_ok(e);
}

toma_status toma_unmerge_weights_export(const toma_desc* desc, const void* w, float* dense, void* stream) {
  Geom g;
  toma_status st = make_geom(desc, &g);
  if (st != TOMA_OK) return st;
  if (!w || !dense) return TOMA_ERR_NULL;
  return cuda_ok(launch_weights_export(merge_geom(g), unmerge_matrix(g, w), dense, (cudaStream_t)stream));
}

}  // extern "C"

namespace toma {
std::atomic<unsigned long long> g_launches{0};
std::atomic<int> g_tune_attention_split{-1}, g_tune_attention_ctas{0}, g_tune_linear_tile{0}, g_tune_block_unfused{0};

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < 64 && (v = cached[dev].load(std::memory_order_relaxed)) > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) return 148;
  if (dev >= 0 && dev < 64) cached[dev].store(v, std::memory_order_relaxed);
  return v;
}
}
extern "C" uint64_t toma_launch_counter(void) { return (uint64_t)toma::g_launches.load(); }

extern "C" void toma_test_set_tuning(int32_t attention_split, int32_t attention_ctas, int32_t linear_tile, int32_t block_unfused) {
  toma::g_tune_block_unfused.store(block_unfused == 1 ? 1 : 0);
  toma::g_tune_attention_split.store(attention_split == 0 || attention_split == 1 ? attention_split : -1);
  toma::g_tune_attention_ctas.store(attention_ctas > 0 ? attention_ctas : 0);
  toma::g_tune_linear_tile.store(linear_tile >= 1 && linear_tile <= 4 ? linear_tile : 0);
}
