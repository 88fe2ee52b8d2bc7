"""ctypes binding of libtoma_b200.so: the same names as the C ABI, argument
marshalling only.  Tensors are torch CUDA tensors; their data pointers and the
current stream handle are passed straight through.  There is no fallback: if the
shared library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int32, c_size_t, c_void_p
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtoma_b200.so")

TOMA_BF16, TOMA_F32 = 0, 1
STATUS_NAMES = ["OK", "ERR_NULL", "ERR_SHAPE", "ERR_DTYPE", "ERR_RATIO", "ERR_TAU", "ERR_WORKSPACE",
                "ERR_UNSUPPORTED", "ERR_CUDA", "ERR_TIMEOUT", "ERR_SCRATCH_LIMIT"]

EXPORTS = ["toma_select_static", "toma_launch_counter", "toma_test_set_tuning", "toma_test_wait_timeout", "toma_workspace_bytes", "toma_weights_bytes", "toma_dest_per_tile", "toma_validate", "toma_status_str",
           "toma_select", "toma_merge_weights", "toma_merge", "toma_attention_workspace_bytes", "toma_attention_plan", "toma_attention",
           "toma_unmerge", "toma_block", "toma_block_host", "toma_linear", "toma_block_proj", "toma_attention_proj_workspace_bytes",
           "toma_attention_proj", "toma_block_mlp", "toma_mlp_workspace_bytes", "toma_mlp",
           "toma_weights_export", "toma_weights_import", "toma_unmerge_weights_export"]

UNMERGE_MODES = {"transpose": 0, "shares": 1}


class TomaDesc(Structure):
    _fields_ = [
        ("batch", c_int32), ("grid_h", c_int32), ("grid_w", c_int32), ("dim", c_int32),
        ("tile_h", c_int32), ("tile_w", c_int32),
        ("merge_ratio", c_float), ("tau", c_float),
        ("reuse_interval", c_int32), ("weight_reuse_interval", c_int32),
        ("n_heads", c_int32), ("head_dim", c_int32), ("n_extra", c_int32), ("dtype", c_int32),
        ("global_merge", c_int32), ("unmerge_mode", c_int32),
    ]


class TomaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: TOMA_{name}")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_10918_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    P = POINTER(TomaDesc)
    lib.toma_workspace_bytes.restype = c_size_t
    lib.toma_workspace_bytes.argtypes = [P]
    lib.toma_weights_bytes.restype = c_size_t
    lib.toma_weights_bytes.argtypes = [P]
    lib.toma_dest_per_tile.restype = c_int32
    lib.toma_dest_per_tile.argtypes = [P]
    lib.toma_launch_counter.restype = ctypes.c_uint64
    lib.toma_launch_counter.argtypes = []
    lib.toma_test_set_tuning.restype = None
    lib.toma_test_set_tuning.argtypes = [c_int32, c_int32, c_int32, c_int32]
    lib.toma_test_wait_timeout.restype = c_int32
    lib.toma_test_wait_timeout.argtypes = [ctypes.c_uint32, c_void_p, c_void_p, c_void_p]
    lib.toma_validate.restype = c_int32
    lib.toma_validate.argtypes = [P]
    lib.toma_status_str.restype = c_char_p
    lib.toma_status_str.argtypes = [c_int32]
    lib.toma_select.restype = c_int32
    lib.toma_select.argtypes = [P, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.toma_select_static.restype = c_int32
    lib.toma_select_static.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.toma_merge_weights.restype = c_int32
    lib.toma_merge_weights.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.toma_merge.restype = c_int32
    lib.toma_merge.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.toma_unmerge.restype = c_int32
    lib.toma_unmerge.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.toma_attention.restype = c_int32
    lib.toma_attention_workspace_bytes.restype = c_size_t
    lib.toma_attention_workspace_bytes.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32]
    lib.toma_attention_plan.restype = c_int32
    lib.toma_attention_plan.argtypes = [c_int32] * 5 + [c_void_p] * 4 + [c_int32]
    lib.toma_attention.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                   c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.toma_block.restype = c_int32
    lib.toma_block.argtypes = [P, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p,
                               c_void_p]
    lib.toma_block_proj.restype = c_int32
    lib.toma_block_proj.argtypes = [P, c_int32] + [c_void_p] * 9 + [c_size_t, c_void_p, c_void_p]
    lib.toma_attention_proj_workspace_bytes.restype = c_size_t
    lib.toma_attention_proj_workspace_bytes.argtypes = [c_int32] * 5
    lib.toma_attention_proj.restype = c_int32
    lib.toma_attention_proj.argtypes = [c_int32] * 5 + [c_void_p] * 7 + [c_size_t, c_void_p, c_void_p]
    lib.toma_block_mlp.restype = c_int32
    lib.toma_block_mlp.argtypes = [P, c_int32, c_void_p, c_void_p, c_void_p, c_int32] + [c_void_p] * 4 + [c_size_t, c_void_p, c_void_p]
    lib.toma_mlp_workspace_bytes.restype = c_size_t
    lib.toma_mlp_workspace_bytes.argtypes = [c_int32] * 4
    lib.toma_mlp.restype = c_int32
    lib.toma_mlp.argtypes = [c_int32] * 4 + [c_void_p] * 5 + [c_size_t, c_void_p, c_void_p]
    lib.toma_linear.restype = c_int32
    lib.toma_linear.argtypes = [c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.toma_block_host.restype = c_int32
    lib.toma_block_host.argtypes = [P, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                    c_size_t, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.toma_weights_export.restype = c_int32
    lib.toma_weights_export.argtypes = [P, c_void_p, c_void_p, c_void_p]
    lib.toma_weights_import.restype = c_int32
    lib.toma_weights_import.argtypes = [P, c_void_p, c_void_p, c_void_p]
    lib.toma_unmerge_weights_export.restype = c_int32
    lib.toma_unmerge_weights_export.argtypes = [P, c_void_p, c_void_p, c_void_p]
    return lib


lib = _load()


def make_desc(*, batch, grid_h, grid_w, dim, tile_h, tile_w, merge_ratio, tau, n_heads, head_dim, dtype,
              reuse_interval=1, weight_reuse_interval=0, n_extra=0, global_merge=False,
              unmerge_mode="transpose") -> TomaDesc:
    code = {"bf16": TOMA_BF16, "f32": TOMA_F32, TOMA_BF16: TOMA_BF16, TOMA_F32: TOMA_F32}[dtype]
    return TomaDesc(batch, grid_h, grid_w, dim, tile_h, tile_w, merge_ratio, tau, reuse_interval,
                    weight_reuse_interval, n_heads, head_dim, n_extra, code, 1 if global_merge else 0,
                    UNMERGE_MODES.get(unmerge_mode, unmerge_mode))


def desc_from_config(cfg, **overrides) -> TomaDesc:
    """Descriptor from a gen.TomaConfig-like object (duck-typed attributes)."""
    kw = dict(batch=cfg.batch, grid_h=cfg.grid_h, grid_w=cfg.grid_w, dim=cfg.dim, tile_h=cfg.tile_h,
              tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio, tau=cfg.tau, n_heads=cfg.n_heads,
              head_dim=cfg.head_dim, dtype=cfg.dtype, reuse_interval=cfg.reuse_interval, n_extra=cfg.n_extra)
    kw.update(overrides)
    return make_desc(**kw)


def torch_dtype(desc: TomaDesc):
    return torch.float32 if desc.dtype == TOMA_F32 else torch.bfloat16


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("tensor must live on a CUDA device (no CPU path exists)")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != 0:
        raise TomaError(status, where)


def toma_validate(desc: TomaDesc) -> int:
    return lib.toma_validate(ctypes.byref(desc))


def toma_workspace_bytes(desc: TomaDesc) -> int:
    return lib.toma_workspace_bytes(ctypes.byref(desc))


def toma_weights_bytes(desc: TomaDesc) -> int:
    return lib.toma_weights_bytes(ctypes.byref(desc))


def toma_test_set_tuning(attention_split: int = -1, attention_ctas: int = 0, linear_tile: int = 0, block_unfused: int = 0) -> None:
    """Test-only: force the attention work plan / the projection tile form / the three-kernel block path
    (defaults restore the library's own choices)."""
    lib.toma_test_set_tuning(attention_split, attention_ctas, linear_tile, block_unfused)


def toma_test_wait_timeout(polls, dev_status, outcome) -> None:
    """Test-only: one CTA waits `polls` polls on a barrier nobody signals, reports through dev_status and returns."""
    _check(lib.toma_test_wait_timeout(polls, _ptr(dev_status), _ptr(outcome), _stream()), "toma_test_wait_timeout")


def toma_dest_per_tile(desc: TomaDesc) -> int:
    return lib.toma_dest_per_tile(ctypes.byref(desc))


def toma_launch_counter() -> int:
    return int(lib.toma_launch_counter())


def toma_status_str(status: int) -> str:
    return lib.toma_status_str(status).decode()


def toma_select(desc, x, idx, ws, dev_status=None):
    _check(lib.toma_select(ctypes.byref(desc), _ptr(x), _ptr(idx), _ptr(ws), ws.numel() * ws.element_size(),
                           _ptr(dev_status), _stream()), "toma_select")


def toma_select_static(desc, x, idx, dev_status=None):
    """toma_select without a workspace argument: the scratch is a fixed array inside the library
    (see include/toma.h for who this is for and what sharing that array implies)."""
    _check(lib.toma_select_static(ctypes.byref(desc), _ptr(x), _ptr(idx), _ptr(dev_status), _stream()),
           "toma_select_static")


def toma_merge_weights(desc, x, idx, w, ws, dev_status=None):
    _check(lib.toma_merge_weights(ctypes.byref(desc), _ptr(x), _ptr(idx), _ptr(w), _ptr(ws),
                                  ws.numel() * ws.element_size(), _ptr(dev_status), _stream()), "toma_merge_weights")


def toma_merge(desc, w, x, xm, dev_status=None):
    _check(lib.toma_merge(ctypes.byref(desc), _ptr(w), _ptr(x), _ptr(xm), _ptr(dev_status), _stream()), "toma_merge")


def toma_unmerge(desc, w, y, out, dev_status=None):
    _check(lib.toma_unmerge(ctypes.byref(desc), _ptr(w), _ptr(y), _ptr(out), _ptr(dev_status), _stream()),
           "toma_unmerge")


def _dtype_code(dtype) -> int:
    return {"bf16": TOMA_BF16, "f32": TOMA_F32, TOMA_BF16: TOMA_BF16, TOMA_F32: TOMA_F32}[dtype]


def toma_attention_workspace_bytes(batch, length, n_heads, head_dim, dtype) -> int:
    return int(lib.toma_attention_workspace_bytes(batch, length, n_heads, head_dim, _dtype_code(dtype)))


def toma_attention_plan(batch, length, n_heads, head_dim, dtype):
    """Work plan of toma_attention for this shape: dict with the CTA count, whether units are split, the
    span bounds and (when split) the owners the kernel's arithmetic gives each span's first and last iteration."""
    cap = 1024
    info = (c_int32 * 4)()
    bounds, first, last = (c_int32 * cap)(), (c_int32 * cap)(), (c_int32 * cap)()
    g = lib.toma_attention_plan(batch, length, n_heads, head_dim, _dtype_code(dtype), info, bounds, first, last, cap)
    if g == 0:
        return None
    return {"ctas": g, "split": bool(info[1]), "units": info[2], "tiles_per_unit": info[3], "bounds": list(bounds[:g + 1]),
            "owner_first": list(first[:g]) if info[1] else None, "owner_last": list(last[:g]) if info[1] else None}


_attention_ws = {}


def toma_attention(batch, length, n_heads, head_dim, dtype, q, k, v, o, dev_status=None, ws=None):
    """ws: scratch tensor of toma_attention_workspace_bytes(); when omitted, one buffer per device is
    kept and grown on demand (callers that overlap attention calls on several streams pass their own)."""
    code = _dtype_code(dtype)
    need = toma_attention_workspace_bytes(batch, length, n_heads, head_dim, code)
    if ws is None and need > 0:
        ws = _attention_ws.get(q.device)
        if ws is None or ws.numel() < need:
            ws = _attention_ws[q.device] = torch.empty(need, dtype=torch.uint8, device=q.device)
    _check(lib.toma_attention(batch, length, n_heads, head_dim, code, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(ws),
                              ws.numel() if ws is not None else 0, _ptr(dev_status), _stream()), "toma_attention")


def toma_block(desc, step, x, out, idx_state, w_state, ws, dev_status=None):
    _check(lib.toma_block(ctypes.byref(desc), step, _ptr(x), _ptr(out), _ptr(idx_state), _ptr(w_state), _ptr(ws),
                          ws.numel() * ws.element_size(), _ptr(dev_status), _stream()), "toma_block")


def toma_linear(a, w, c, dev_status=None):
    """c = a @ w for 2-D tensors a [m, k], w [k, n], c [m, n] of the same dtype (bf16 or fp32)."""
    m, k = a.shape
    n = w.shape[1]
    code = TOMA_F32 if a.dtype == torch.float32 else TOMA_BF16
    _check(lib.toma_linear(m, n, k, code, _ptr(a), _ptr(w), _ptr(c), _ptr(dev_status), _stream()), "toma_linear")


def toma_block_proj(desc, step, x, wq, wk, wv, wo, out, idx_state, w_state, ws, dev_status=None):
    _check(lib.toma_block_proj(ctypes.byref(desc), step, _ptr(x), _ptr(wq), _ptr(wk), _ptr(wv), _ptr(wo), _ptr(out),
                               _ptr(idx_state), _ptr(w_state), _ptr(ws), ws.numel() * ws.element_size(), _ptr(dev_status),
                               _stream()), "toma_block_proj")


def toma_attention_proj_workspace_bytes(batch, length, n_heads, head_dim, dtype) -> int:
    return int(lib.toma_attention_proj_workspace_bytes(batch, length, n_heads, head_dim, _dtype_code(dtype)))


def toma_attention_proj(batch, length, n_heads, head_dim, dtype, x, wq, wk, wv, wo, out, ws, dev_status=None):
    _check(lib.toma_attention_proj(batch, length, n_heads, head_dim, _dtype_code(dtype), _ptr(x), _ptr(wq), _ptr(wk),
                                   _ptr(wv), _ptr(wo), _ptr(out), _ptr(ws), ws.numel() * ws.element_size(),
                                   _ptr(dev_status), _stream()), "toma_attention_proj")


def toma_block_mlp(desc, step, x, w1, w2, out, idx_state, w_state, ws, dev_status=None):
    """w1 [dim][hidden], w2 [hidden][dim]; hidden is read from w1's shape."""
    hidden = int(w1.shape[1])
    _check(lib.toma_block_mlp(ctypes.byref(desc), step, _ptr(x), _ptr(w1), _ptr(w2), hidden, _ptr(out), _ptr(idx_state),
                              _ptr(w_state), _ptr(ws), ws.numel() * ws.element_size(), _ptr(dev_status), _stream()),
           "toma_block_mlp")


def toma_mlp_workspace_bytes(rows, dim, hidden, dtype) -> int:
    return int(lib.toma_mlp_workspace_bytes(rows, dim, hidden, _dtype_code(dtype)))


def toma_mlp(rows, dim, hidden, dtype, x, w1, w2, out, ws, dev_status=None):
    _check(lib.toma_mlp(rows, dim, hidden, _dtype_code(dtype), _ptr(x), _ptr(w1), _ptr(w2), _ptr(out), _ptr(ws),
                        ws.numel() * ws.element_size(), _ptr(dev_status), _stream()), "toma_mlp")


def toma_block_host(desc, step, x_host, out_host, x_dev, out_dev, idx_state, w_state, ws, dev_status=None,
                    copy_in_stream=None, copy_out_stream=None, copied_in_event=None, computed_event=None):
    """x_host / out_host: CPU tensors (pinned for asynchronous copies); the streams are torch.cuda.Stream
    objects and the events torch.cuda.Event objects that have been recorded at least once (so that
    their handles exist), or None to run everything on the current stream."""
    if x_host.is_cuda or out_host.is_cuda:
        raise ValueError("toma_block_host takes host tensors for x_host / out_host")

    def handle(obj, attr):
        return None if obj is None else getattr(obj, attr)

    _check(lib.toma_block_host(ctypes.byref(desc), step, x_host.data_ptr(), out_host.data_ptr(), _ptr(x_dev),
                               _ptr(out_dev), _ptr(idx_state), _ptr(w_state), _ptr(ws), ws.numel() * ws.element_size(),
                               _ptr(dev_status), _stream(), handle(copy_in_stream, "cuda_stream"),
                               handle(copy_out_stream, "cuda_stream"), handle(copied_in_event, "cuda_event"),
                               handle(computed_event, "cuda_event")), "toma_block_host")


def toma_weights_export(desc, w, dense):
    _check(lib.toma_weights_export(ctypes.byref(desc), _ptr(w), _ptr(dense), _stream()), "toma_weights_export")


def toma_unmerge_weights_export(desc, w, dense):
    _check(lib.toma_unmerge_weights_export(ctypes.byref(desc), _ptr(w), _ptr(dense), _stream()),
           "toma_unmerge_weights_export")


def toma_weights_import(desc, dense, w):
    _check(lib.toma_weights_import(ctypes.byref(desc), _ptr(dense), _ptr(w), _stream()), "toma_weights_import")


# ---- allocation helpers (torch owns the memory; the library never allocates) ----

def alloc_workspace(desc, device="cuda") -> torch.Tensor:
    return torch.empty(max(toma_workspace_bytes(desc), 16), dtype=torch.uint8, device=device)


def alloc_weights(desc, device="cuda") -> torch.Tensor:
    return torch.empty(max(toma_weights_bytes(desc), 16), dtype=torch.uint8, device=device)


def alloc_idx(desc, device="cuda") -> torch.Tensor:
    tiles = (desc.grid_h // desc.tile_h) * (desc.grid_w // desc.tile_w)
    return torch.empty((desc.batch, tiles, toma_dest_per_tile(desc)), dtype=torch.int32, device=device)
