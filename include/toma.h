/*
 * toma.h -- C ABI of the B200 (sm_100a) ToMA token-reduction library.
 *
 * The library implements, per transformer block, the locality-aware ToMA path
 * of "ToMA: Token Merge with Attention for Diffusion Models" (Algorithm 3):
 * split the H x W token grid into equal tiles, pick destination tokens in every
 * tile by greedy facility-location maximisation (Algorithm 2), build the
 * attention-like merge weights (Sec. 4.2.1), merge N tokens to D, run the core
 * attention over the D merged tokens (Eq. 1), and unmerge with the transposed
 * weights (Sec. 4.2.2).  Selection and weights are reused between refresh
 * steps (Sec. 4.3.2).
 *
 * Conventions that hold for every entry point
 *   - Every data pointer is DEVICE memory owned by the caller, 16-byte aligned,
 *     dense row-major.  `desc` is HOST memory.  The library never allocates,
 *     frees or synchronises; work is enqueued on `stream` (a cudaStream_t
 *     passed as void*; NULL is the default stream).
 *   - Errors the host can detect (null pointers, shapes that do not divide,
 *     unsupported sizes, a workspace that is too small) are returned before
 *     anything is launched.  Conditions only the device can see (a bounded wait
 *     inside a kernel that ran out) are OR-ed into `*dev_status`, a caller-owned
 *     device word that the caller zeroes and reads after synchronising; the
 *     kernels still exit cleanly.  `dev_status` may be NULL.
 *   - There is no CPU fallback: without a CUDA device the calls fail with
 *     TOMA_ERR_CUDA.
 *
 * Token layout.  X is [batch][grid_h*grid_w + n_extra][dim].  Image token
 * n = y*grid_w + x lies in tile p = (y/tile_h)*(grid_w/tile_w) + x/tile_w at
 * local slot l = (y%tile_h)*tile_w + x%tile_w.  N_loc = tile_h*tile_w,
 * P = tiles per image, D_loc = N_loc - round(merge_ratio*N_loc) destinations
 * per tile, D = P*D_loc.  Merged tensors are [batch][D + n_extra][dim] with row
 * p*D_loc + k holding destination k (greedy pick order) of tile p; the n_extra
 * trailing (text) tokens are never merged and follow the D merged rows.
 */
#ifndef TOMA_H_
#define TOMA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define TOMA_API __attribute__((visibility("default")))
#else
#define TOMA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TOMA_OK = 0,
  TOMA_ERR_NULL = 1,        /* a required pointer is NULL */
  TOMA_ERR_SHAPE = 2,       /* tiles do not divide the grid, dim not a multiple of 8, heads*head_dim != dim ... */
  TOMA_ERR_DTYPE = 3,
  TOMA_ERR_RATIO = 4,       /* merge_ratio outside [0,1) or leaving no destination */
  TOMA_ERR_TAU = 5,         /* tau <= 0 or not finite */
  TOMA_ERR_WORKSPACE = 6,   /* workspace missing or smaller than toma_workspace_bytes() */
  TOMA_ERR_UNSUPPORTED = 7, /* N_loc > 1024, head_dim not 64/128 in bf16 mode, dim > 4096 ... */
  TOMA_ERR_CUDA = 8,        /* a CUDA runtime call or launch failed */
  TOMA_ERR_TIMEOUT = 9,     /* only ever reported through *dev_status (bit 0) */
  TOMA_ERR_SCRATCH_LIMIT = 10 /* toma_select_static: the problem needs more than TOMA_STATIC_SCRATCH_BYTES */
} toma_status;

/* Size of the fixed scratch array built into the library for toma_select_static (16 MiB). */
#define TOMA_STATIC_SCRATCH_BYTES (16u << 20)

typedef enum { TOMA_BF16 = 0, TOMA_F32 = 1 } toma_dtype;

/* Problem statement of Algorithm 3 (token tensor shape, region layout, merge
 * ratio, temperature) plus the reuse schedule of Sec. 4.3.2.  Plain data. */
typedef struct {
  int32_t batch, grid_h, grid_w, dim;
  int32_t tile_h, tile_w;          /* must divide grid_h / grid_w; a stripe is tile_h x grid_w */
  float merge_ratio;               /* fraction of tokens REMOVED, in [0, 1) */
  float tau;                       /* merge temperature; logits are <d_i, x_k> / (tau * sqrt(dim)) */
  int32_t reuse_interval;          /* k >= 1: toma_block refreshes selection when step % k == 0 */
  int32_t weight_reuse_interval;   /* 0: same as reuse_interval; else weights are refreshed when
                                      step % weight_reuse_interval == 0 from the cached selection */
  int32_t n_heads, head_dim;       /* n_heads*head_dim == dim (attention inside toma_block) */
  int32_t n_extra;                 /* trailing un-merged tokens */
  int32_t dtype;                   /* toma_dtype of x / merged / out tensors */
  int32_t global_merge;            /* 0: weights, merge and unmerge per tile (Algorithm 3).  1: destinations are
                                      still chosen per tile, but the D destinations of an image form one set and
                                      weights, merge and unmerge run over all N image tokens (the paper's default
                                      variant, Sec. 5).  Merged rows keep the tile-major pick order; the weight
                                      buffer then holds A~^T as [batch][N][D] and is far larger */
  int32_t unmerge_mode;            /* matrix toma_unmerge applies (Sec. 4.2.2): TOMA_UNMERGE_TRANSPOSE (0), the
                                      transpose A~^T of the merge weights, Algorithm 3's choice;
                                      TOMA_UNMERGE_SHARES (1), the transpose A^T of the column-stochastic
                                      softmax matrix before its rows are normalised: every source token gets
                                      the convex combination of the destinations' outputs given by its own
                                      softmax shares, so a constant input comes back unchanged.  A non-zero mode
                                      keeps a second matrix in the weight buffer (twice the size) */
} toma_desc;

enum { TOMA_UNMERGE_TRANSPOSE = 0, TOMA_UNMERGE_SHARES = 1 };

/* Host-only helpers.  Return 0 / negative on an invalid descriptor. */
TOMA_API size_t toma_workspace_bytes(const toma_desc* desc);   /* scratch needed by select / merge_weights / block */
TOMA_API size_t toma_weights_bytes(const toma_desc* desc);     /* size of one weight buffer `w` */
TOMA_API int32_t toma_dest_per_tile(const toma_desc* desc);    /* D_loc */
TOMA_API toma_status toma_validate(const toma_desc* desc);
TOMA_API const char* toma_status_str(toma_status s);
/* Total number of kernels this library has launched in this process (monotonic; for benchmarks). */
TOMA_API uint64_t toma_launch_counter(void);
/* TEST-ONLY: overrides launch heuristics so that the parity tests can drive every code path of the
 * attention kernel's work plan (Eq. 1) and every tile form of the projection kernel (App. C's 4 d^2 N
 * term).  The library itself never calls it and reads no environment variable; results do not depend
 * on these settings, only the launch configuration does.  Process-wide; not for concurrent use.
 *   attention_split: 0 = whole work units per CTA, 1 = spans cut at single key tiles, other = heuristic
 *   attention_ctas : > 0 = number of persistent CTAs (clamped to the scratch capacity), else heuristic
 *   linear_tile    : 1 = 128 x 256, 2 = 128 x 320, 3 = 256 x 256, 4 = 128 x 128 tiles, else heuristic
 *   block_unfused  : 1 = toma_block runs merge, attention and unmerge as three kernels even for the shapes its
 *                    one-kernel reuse step covers, selection and weights of 64-token tiles as their separate
 *                    kernels instead of one, and the weights of large tiles through the gather and the logits
 *                    contraction instead of out of the raw Gram matrix (so that both paths can be compared), else
 *                    the library chooses */
TOMA_API void toma_test_set_tuning(int32_t attention_split, int32_t attention_ctas, int32_t linear_tile,
                                   int32_t block_unfused);
/* TEST-ONLY (no counterpart in the paper): launches one CTA that waits, with the library's bounded wait and
 * a limit of `polls` polls (1..100000), on a barrier that nobody signals.  The wait gives up, ORs
 * TOMA_ERR_TIMEOUT's bit (bit 0) into *dev_status (device, may be NULL), writes 2 to *outcome (device, may be
 * NULL; 1 would mean the wait completed) and the kernel returns: nothing traps, faults or spins without
 * limit, and the context stays usable.  This is the path every device-side wait of the library takes when
 * its producer never comes. */
TOMA_API toma_status toma_test_wait_timeout(uint32_t polls, uint32_t* dev_status, uint32_t* outcome, void* stream);

/* Destination selection (Sec. 4.1, Algorithm 2) inside every tile.
 *   x   [batch][N + n_extra][dim]  in
 *   idx [batch][P][D_loc] int32    out: tile-local indices (0..N_loc-1) in greedy pick order
 * Similarity is the fixed-point cosine: each token is scaled to length 0.99,
 * quantised to a bf16-representable grid of 2^-12 steps, the Gram matrix is
 * accumulated exactly and rounded to int16 units of 2^-12 (diagonal forced to
 * 4014).  Gains are exact integers; ties go to the lowest index; selected
 * tokens are excluded from later rounds.  Uses `ws` as scratch. */
TOMA_API toma_status toma_select(const toma_desc* desc, const void* x, int32_t* idx, void* ws, size_t ws_bytes,
                        uint32_t* dev_status, void* stream);

/* toma_select for callers that have no workspace to give and may not allocate one.
 * (No counterpart in the paper: this exists for integration, not for the method.)
 * Meant for code that only receives its tensors and a stream -- a runtime's per-layer hook, a
 * plug-in inside another program's step loop -- where cudaMalloc is off the table because it
 * synchronises the device, is illegal during stream capture and sidesteps the host's memory pool.
 * Same inputs, outputs and results as toma_select; the scratch is a static device array of
 * TOMA_STATIC_SCRATCH_BYTES inside the library, so:
 *   - a GPU holds that much memory from the moment the library's device code is loaded on it (with the
 *     CUDA runtime's default lazy loading: from the first toma_select_static call on that GPU) until
 *     process exit;
 *   - a problem whose scratch, batch*P*N_loc*(dim + N_loc)*2 bytes plus padding, exceeds it is
 *     refused with TOMA_ERR_SCRATCH_LIMIT before any launch;
 *   - all calls on a device share it and it keeps the previous call's contents (nothing needs
 *     zeroing: every byte read is written earlier in the same call); calls that can overlap on
 *     the GPU race on it, so the caller must serialise them;
 *   - the first call on each device resolves the array's device address, which is also where the
 *     memory is reserved: it returns TOMA_ERR_CUDA (nothing launched, no sticky error left) if the
 *     device has none left; make that call before starting any stream capture.
 * The call never allocates or frees memory. */
TOMA_API toma_status toma_select_static(const toma_desc* desc, const void* x, int32_t* idx, uint32_t* dev_status,
                                        void* stream);

/* Merge weights (Sec. 4.2.1).  For each tile: logits between the D_loc selected
 * tokens and all N_loc tokens, softmax over the destination axis per source
 * token, then each destination row normalised to sum 1.
 *   w: opaque buffer of toma_weights_bytes(); holds A~^T per tile as [N_loc][D_loc].  In f32
 *      mode one fp32 plane per tile; in bf16 mode two bf16 planes per tile, [2][N_loc][D_loc],
 *      the weight rounded to bf16 and the bf16-rounded remainder, whose sum carries 16
 *      significant bits.  Read it back as fp32 with toma_weights_export.  Uses `ws` as scratch. */
TOMA_API toma_status toma_merge_weights(const toma_desc* desc, const void* x, const int32_t* idx, void* w, void* ws,
                               size_t ws_bytes, uint32_t* dev_status, void* stream);

/* Merge X_m = A~ X per tile (Sec. 4.2.1).  xm [batch][D + n_extra][dim] out; extra tokens copied. */
TOMA_API toma_status toma_merge(const toma_desc* desc, const void* w, const void* x, void* xm, uint32_t* dev_status,
                       void* stream);

/* Scratch bytes toma_attention needs for this shape (0 when the shape's kernel needs none, or
 * when an argument is invalid).  Host-only. */
TOMA_API size_t toma_attention_workspace_bytes(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim,
                                               int32_t dtype);

/* Host-only diagnostic: how toma_attention would cut this shape's work across its persistent CTAs.
 * A work unit is (batch, head, 256 queries); an iteration is one 64-key tile of a unit; CTA g runs the
 * iterations bounds[g] .. bounds[g+1]-1 of the units laid end to end.
 *   info[0] = number of CTAs G, info[1] = 1 if units are split between CTAs (cut at single key
 *   tiles) or 0 if every CTA gets whole units, info[2] = work units, info[3] = key tiles per unit.
 *   bounds (NULL or >= min(G+1, capacity) entries), owner_first / owner_last (NULL or >= min(G, capacity)
 *   entries; filled only when units are split): the CTA the kernel's own arithmetic assigns to the
 *   first and to the last iteration of span g (both equal g).
 * Returns G, or 0 when the shape does not run on the tensor-core kernel (fp32, head_dim not 64/128). */
TOMA_API int32_t toma_attention_plan(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype,
                                     int32_t info[4], int32_t* bounds, int32_t* owner_first, int32_t* owner_last,
                                     int32_t capacity);

/* Multi-head attention core softmax(Q K^T / sqrt(head_dim)) V (Eq. 1 with tau = 1), no mask.
 *   q, k, v, o: [batch][len][n_heads][head_dim], device.
 *   ws: device scratch of at least toma_attention_workspace_bytes(), 16-byte aligned, caller-owned,
 *       no initialisation needed; may be NULL when that size is 0.  The call's kernels write it, so
 *       calls that can overlap on the GPU need separate scratch.  TOMA_ERR_WORKSPACE otherwise. */
TOMA_API toma_status toma_attention(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype,
                           const void* q, const void* k, const void* v, void* o, void* ws, size_t ws_bytes,
                           uint32_t* dev_status, void* stream);

/* Unmerge out = A~^T y per tile, written back in spatial order (Sec. 4.2.2, Algorithm 3 step 3).
 *   y [batch][D + n_extra][dim] in; out [batch][N + n_extra][dim]; extra tokens copied. */
TOMA_API toma_status toma_unmerge(const toma_desc* desc, const void* w, const void* y, void* out, uint32_t* dev_status,
                         void* stream);

/* Dense projection c = a w: the linear maps of the wrapped module (the Q/K/V and output projections of
 * attention, whose cost App. C counts as the 4 d^2 N term that shrinks with the merged length).
 *   a [m][k], w [k][n], c [m][n]: device, row-major, dense, 16-byte aligned; bf16 needs n and k
 *   multiples of 8.  bf16 runs on the tensor cores with fp32 accumulation, fp32 on FFMA. */
TOMA_API toma_status toma_linear(int32_t m, int32_t n, int32_t k, int32_t dtype, const void* a, const void* w, void* c,
                                 uint32_t* dev_status, void* stream);

/* One ToMA-wrapped attention call (Algorithm 3) with pattern reuse (Sec. 4.3.2):
 * refresh idx_state / w_state when the schedule says so, then merge, attention
 * with Q = K = V = merged tokens, unmerge.  idx_state [batch][P][D_loc] and
 * w_state (toma_weights_bytes()) persist between calls and are caller-owned. */
TOMA_API toma_status toma_block(const toma_desc* desc, int32_t step, const void* x, void* out, int32_t* idx_state,
                       void* w_state, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream);

/* toma_block with the whole attention module as the wrapped F (Algorithm 3 applies F to the merged tokens,
 * so the module's projections shrink with them): Q = X_m wq, K = X_m wk, V = X_m wv, attention, then wo,
 * then the unmerge.  wq, wk, wv, wo: [dim][dim] row-major [in][out], device, dtype of x.  Everything else as
 * toma_block (same workspace size). */
TOMA_API toma_status toma_block_proj(const toma_desc* desc, int32_t step, const void* x, const void* wq, const void* wk,
                                     const void* wv, const void* wo, void* out, int32_t* idx_state, void* w_state, void* ws,
                                     size_t ws_bytes, uint32_t* dev_status, void* stream);

/* The same attention module on all tokens, without ToMA: out = attention(x wq, x wk, x wv) wo.  The
 * full-token baseline of toma_block_proj.  x, out [batch][len][n_heads*head_dim];
 * ws: device scratch of toma_attention_proj_workspace_bytes(), 16-byte aligned. */
TOMA_API size_t toma_attention_proj_workspace_bytes(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim,
                                                    int32_t dtype);
TOMA_API toma_status toma_attention_proj(int32_t batch, int32_t len, int32_t n_heads, int32_t head_dim, int32_t dtype,
                                         const void* x, const void* wq, const void* wk, const void* wv, const void* wo,
                                         void* out, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream);

/* toma_block with the MLP as the wrapped F (Sec. 4.2.2: the merged tokens go through "Attention/MLP"):
 * merge, H = GELU(X_m w1), Y = H w2, unmerge.  GELU(v) = v Phi(v) with the exact normal distribution
 * function (erf), applied to the fp32 accumulator before H is stored in the dtype of x.
 *   w1 [dim][hidden], w2 [hidden][dim]: row-major [in][out], device, dtype of x, no biases;
 *   hidden: a multiple of 8, at most 4 * dim (H lives in the block's workspace).  TOMA_ERR_SHAPE otherwise.
 * Everything else as toma_block (same workspace size; n_heads / head_dim are validated but unused). */
TOMA_API toma_status toma_block_mlp(const toma_desc* desc, int32_t step, const void* x, const void* w1, const void* w2,
                                    int32_t hidden, void* out, int32_t* idx_state, void* w_state, void* ws, size_t ws_bytes,
                                    uint32_t* dev_status, void* stream);

/* The same MLP on all rows, without ToMA: out = GELU(x w1) w2, x and out [rows][dim].  The full-token baseline
 * of toma_block_mlp.  ws: device scratch of toma_mlp_workspace_bytes() (the hidden tensor), 16-byte aligned;
 * bf16 needs dim and hidden multiples of 8. */
TOMA_API size_t toma_mlp_workspace_bytes(int32_t rows, int32_t dim, int32_t hidden, int32_t dtype);
TOMA_API toma_status toma_mlp(int32_t rows, int32_t dim, int32_t hidden, int32_t dtype, const void* x, const void* w1,
                              const void* w2, void* out, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream);

/* toma_block for callers whose tokens live in HOST memory (Algorithm 3 end to end, copies included):
 * copy x_host -> x_dev, run toma_block(x_dev -> out_dev), copy out_dev -> out_host.
 *   x_host, out_host: HOST buffers of batch*(N + n_extra)*dim elements, caller-owned.  Page-locked
 *       memory makes the copies asynchronous; pageable memory works but the copies then block the host.
 *   x_dev, out_dev: DEVICE staging buffers of the same size, caller-owned (the library never allocates).
 *   stream: where the block's kernels run.  copy_in_stream / copy_out_stream: where the two copies
 *       run; NULL means `stream` (everything in order on one stream).  With separate streams the call
 *       chains copy-in -> kernels -> copy-out through the two caller-owned events (cudaEvent_t passed
 *       as void*, required in that case), so that the copies of neighbouring steps overlap this step's
 *       kernels.  The caller then orders what the call cannot see: a staging buffer may be handed to a
 *       later call only after the earlier call's use of it has finished.
 * Errors as toma_block; TOMA_ERR_NULL if separate streams are given without events. */
TOMA_API toma_status toma_block_host(const toma_desc* desc, int32_t step, const void* x_host, void* out_host, void* x_dev,
                                     void* out_dev, int32_t* idx_state, void* w_state, void* ws, size_t ws_bytes,
                                     uint32_t* dev_status, void* stream, void* copy_in_stream, void* copy_out_stream,
                                     void* copied_in_event, void* computed_event);

/* Conversions between the opaque weight buffer and dense fp32 A~ [batch][P][D_loc][N_loc]
 * (device pointers).  For tests and for callers that bring their own weights (a
 * one-hot matrix makes merge a hard ToMeSD-style merge, Sec. 4.2). */
TOMA_API toma_status toma_weights_export(const toma_desc* desc, const void* w, float* dense, void* stream);
TOMA_API toma_status toma_weights_import(const toma_desc* desc, const float* dense, void* w, void* stream);
/* The matrix toma_unmerge applies, transposed back to dense fp32 [batch][P][D_loc][N_loc]: A~ itself with
 * TOMA_UNMERGE_TRANSPOSE, the second matrix of the weight buffer otherwise.  With a non-zero unmerge_mode
 * toma_weights_import fills both matrices with `dense`. */
TOMA_API toma_status toma_unmerge_weights_export(const toma_desc* desc, const void* w, float* dense, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TOMA_H_ */
