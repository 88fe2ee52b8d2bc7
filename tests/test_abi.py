"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and
rejects bad descriptors before launching anything.  No compute calls (no GPU needed)."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def toma():
    entry.build()
    import paper_2509_10918_b200 as t
    return t


def test_every_declared_symbol_is_exported(toma):
    header = open(os.path.join(ROOT, "include", "toma.h")).read()
    declared = set(re.findall(r"TOMA_API[^;(]*?\b(toma_\w+)\s*\(", header))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(toma.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared but not exported"
    assert declared == set(toma.EXPORTS)


def test_binding_declares_argument_types_for_every_entry_point(toma):
    # without argtypes ctypes passes a Python int as a 32-bit C int and a device pointer loses its upper half
    for name in toma.EXPORTS:
        assert getattr(toma.lib, name).argtypes is not None, f"{name}: ctypes argtypes not declared"


def _desc(toma, **kw):
    base = dict(batch=2, grid_h=64, grid_w=64, dim=640, tile_h=16, tile_w=16, merge_ratio=0.5, tau=0.1, n_heads=10,
                head_dim=64, dtype="bf16")
    base.update(kw)
    return toma.make_desc(**base)


def test_descriptor_validation(toma):
    OK, SHAPE, DTYPE, RATIO, TAU, UNSUP = 0, 2, 3, 4, 5, 7
    assert toma.toma_validate(_desc(toma)) == OK
    assert toma.toma_validate(_desc(toma, tile_h=24)) == SHAPE          # does not divide the grid
    assert toma.toma_validate(_desc(toma, dim=644, n_heads=7, head_dim=92)) == SHAPE  # dim % 8
    assert toma.toma_validate(_desc(toma, n_heads=9)) == SHAPE
    assert toma.toma_validate(_desc(toma, merge_ratio=1.0)) == RATIO
    assert toma.toma_validate(_desc(toma, merge_ratio=-0.1)) == RATIO
    assert toma.toma_validate(_desc(toma, merge_ratio=0.999)) == RATIO   # leaves no destination
    assert toma.toma_validate(_desc(toma, tau=0.0)) == TAU
    assert toma.toma_validate(_desc(toma, tau=float("nan"))) == TAU
    assert toma.toma_validate(_desc(toma, tile_h=64, tile_w=32)) == UNSUP  # N_loc = 2048
    assert toma.toma_validate(_desc(toma, reuse_interval=0)) == SHAPE
    d = _desc(toma)
    d.dtype = 5
    assert toma.toma_validate(d) == DTYPE
    assert toma.toma_validate(_desc(toma, unmerge_mode="shares")) == OK
    assert toma.toma_validate(_desc(toma, unmerge_mode=2)) == SHAPE
    assert toma.toma_validate(_desc(toma, unmerge_mode=-1)) == SHAPE


def test_sizes(toma):
    d = _desc(toma)
    assert toma.toma_dest_per_tile(d) == 128
    assert toma.toma_weights_bytes(d) == 2 * 16 * 256 * 128 * 4  # hi + lo bf16 planes
    assert toma.toma_weights_bytes(_desc(toma, unmerge_mode="shares")) == 2 * toma.toma_weights_bytes(d)  # A~^T and A^T
    assert toma.toma_workspace_bytes(d) > 0
    assert toma.toma_dest_per_tile(_desc(toma, merge_ratio=0.25)) == 192
    assert toma.toma_dest_per_tile(_desc(toma, merge_ratio=0.75)) == 64
    assert toma.toma_workspace_bytes(_desc(toma, tau=-1.0)) == 0
    assert toma.toma_status_str(6).startswith("workspace")


def test_null_and_workspace_errors_are_returned_before_any_launch(toma):
    d = _desc(toma)
    lib = toma.lib
    NULL, WS = 1, 6
    assert lib.toma_select(ctypes.byref(d), None, None, None, 0, None, None) == NULL
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    assert lib.toma_select(ctypes.byref(d), fake, fake, None, 0, None, None) == WS
    assert lib.toma_select(ctypes.byref(d), fake, fake, fake, 16, None, None) == WS
    assert lib.toma_merge(ctypes.byref(d), None, fake, fake, None, None) == NULL
    assert lib.toma_attention(1, 0, 1, 64, 0, fake, fake, fake, fake, None, 0, None, None) == 2
    assert lib.toma_attention(1, 8, 1, 48, 0, fake, fake, fake, fake, None, 0, None, None) == 7
    # the tensor-core attention needs scratch: missing or short scratch is refused before any launch
    need = lib.toma_attention_workspace_bytes(2, 2048, 10, 64, 0)
    assert need > 0 and lib.toma_attention_workspace_bytes(2, 2048, 10, 64, 1) == 0  # fp32 path needs none
    assert lib.toma_attention(2, 2048, 10, 64, 0, fake, fake, fake, fake, None, 0, None, None) == WS
    assert lib.toma_attention(2, 2048, 10, 64, 0, fake, fake, fake, fake, fake, need - 1, None, None) == WS
    assert lib.toma_block_host(ctypes.byref(d), 0, None, fake, fake, fake, fake, fake, fake, 1 << 40, None, None, None,
                               None, None, None) == NULL
    # separate copy streams without the events that chain them
    assert lib.toma_block_host(ctypes.byref(d), 0, fake, fake, fake, fake, fake, fake, fake, 1 << 40, None, None, fake,
                               None, None, None) == NULL


def test_destinations_per_tile_agree_with_the_oracle_on_every_config(toma):
    """The library's D_loc (toma_dest_per_tile) and the oracle's (dest_count) are computed independently; the
    buffers of the GPU tests are sized from the former, the expected values from the latter."""
    import gen
    from oracle import toma_oracle as O
    for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5a", "cfg5b"):
        for ratio in (None, 0.25, 0.75, 0.3, 0.99, 0.0):
            cfg = gen.config(name) if ratio is None else gen.config(name, merge_ratio=ratio)
            assert toma.toma_dest_per_tile(toma.desc_from_config(cfg)) == O.dest_count(cfg.n_loc, cfg.merge_ratio)


def test_binding_refuses_cpu_tensors(toma):
    import torch
    d = _desc(toma)
    x = torch.zeros(4)
    with pytest.raises(ValueError):
        toma.toma_merge(d, x, x, x)


@pytest.mark.parametrize("split", ["0", "1", None])
@pytest.mark.parametrize("shape", [(2, 2048, 10, 64), (1, 2560, 24, 128), (2, 1000, 3, 64), (1, 77, 2, 128),
                                   (4, 8192, 10, 64), (1, 300, 3, 64), (3, 4096, 7, 64)])
def test_attention_work_plan_covers_every_key_tile_once(toma, shape, split):
    """Host logic of the attention kernel's work plan (no GPU needed): the spans tile the iteration space
    [0, units * tiles_per_unit) without gap or overlap, differ by at most one quantum, keep units whole
    when the plan says so, and the kernel's own owner arithmetic maps each span's ends back to its CTA."""
    B, L, h, dh = shape
    toma.toma_test_set_tuning(attention_split=-1 if split is None else int(split))
    try:
        plan = toma.toma_attention_plan(B, L, h, dh, "bf16")
    finally:
        toma.toma_test_set_tuning()
    units, nblk = B * h * ((L + 255) // 256), (L + 63) // 64
    assert plan["units"] == units and plan["tiles_per_unit"] == nblk
    b = plan["bounds"]
    assert len(b) == plan["ctas"] + 1 and b[0] == 0 and b[-1] == units * nblk
    sizes = [b[g + 1] - b[g] for g in range(plan["ctas"])]
    assert min(sizes) >= 1
    if split is not None:
        assert plan["split"] == (split == "1")
    if plan["split"] and (units * nblk) // plan["ctas"] >= 2 * nblk:
        # long spans: equal to within one tile, then bounds within two tiles of a unit boundary are moved onto it
        assert max(sizes) - min(sizes) <= 1 + 2 * 2
        for x in b[1:-1]:
            off = min(x % nblk, nblk - x % nblk)
            assert off == 0 or off > 2, "a bound sits within two tiles of a unit boundary"
        assert plan["owner_first"] == list(range(plan["ctas"])) and plan["owner_last"] == list(range(plan["ctas"]))
    elif plan["split"]:
        # short spans: the longest span, charged 2 per key tile plus 4 per whole-unit piece and 8 per partial piece
        # (half tiles), is as short as a left-to-right cut into at most 148 spans can make it
        def cost(lo, hi):
            c, it = 0, lo
            while it < hi:
                end = min(hi, (it // nblk + 1) * nblk)
                c += 2 * (end - it) + (4 if (it % nblk == 0 and end % nblk == 0) else 8)
                it = end
            return c

        def spans_needed(budget):
            n, it, T = 0, 0, units * nblk
            while it < T:
                end = it
                while end < T:
                    # one more tile - or, where that is too dear, on to the end of the unit: completing a unit that
                    # the span entered at its first tile makes the piece a whole one, which is cheaper
                    edge = min(T, (end // nblk + 1) * nblk)
                    if cost(it, end + 1) <= budget:
                        end += 1
                    elif cost(it, edge) <= budget:
                        end = edge
                    else:
                        break
                if end == it:
                    return None
                n, it = n + 1, end
            return n

        worst = max(cost(b[g], b[g + 1]) for g in range(plan["ctas"]))
        assert plan["ctas"] <= 148
        fewer = spans_needed(worst - 1)
        assert fewer is None or fewer > 148, "a smaller budget would have done"
        assert plan["owner_first"] == list(range(plan["ctas"])) and plan["owner_last"] == list(range(plan["ctas"]))
    else:
        assert all(x % nblk == 0 for x in b) and max(sizes) - min(sizes) <= nblk
    assert toma.toma_attention_plan(B, L, h, dh, "f32") is None
