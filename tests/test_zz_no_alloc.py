"""toma_select_static: the selection entry point for callers that may not allocate.

Some integrations (a runtime's layer hook, a plug-in in another program's step loop) get only
tensors and a stream: they have no workspace to pass and cannot call cudaMalloc where they run.
For them the library keeps the selection scratch in a fixed static device array.  This test calls
that entry point through the C ABI twice in a row, on different inputs, and requires exactly the
indices the workspace-taking toma_select produces (selection is integer work: bit-exact), so a
second call that tripped over the first call's leftovers in the shared array would show.  It is
collected last so that a run stopping at the first failure has already exercised everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

import gen
from tests._util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def toma():
    import __graft_entry__ as entry
    entry.build()
    import paper_2509_10918_b200 as t
    return t


def _reference_select(toma, desc, x):
    idx = toma.alloc_idx(desc)
    ws = toma.alloc_workspace(desc)
    toma.toma_select(desc, x, idx, ws)
    torch.cuda.synchronize()
    return idx.cpu().numpy()


def test_static_scratch_select_matches_workspace_select_twice(toma):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # two different problems back to back: the second is smaller, so it runs inside memory the
    # first call filled
    for name, over in (("cfg3", {}), ("cfg2", {}), ("cfg3", {"seed": 3})):
        cfg = gen.config(name, **over)
        desc = toma.desc_from_config(cfg)
        x = to_dev(gen.features(cfg), cfg.dtype)
        want = _reference_select(toma, desc, x)
        got = toma.alloc_idx(desc)
        got.fill_(-1)
        toma.toma_select_static(desc, x, got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(got.cpu().numpy(), want), f"static-scratch selection differs on {name}"


def test_static_scratch_rejects_oversized_problems(toma):
    cfg = gen.config("cfg5a")  # 256 tiles x 256 tokens x 640 channels: far beyond 16 MiB of scratch
    desc = toma.desc_from_config(cfg)
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: the size check comes before any launch
    SCRATCH_LIMIT = 10
    assert toma.lib.toma_select_static(ctypes.byref(desc), fake, fake, None, None) == SCRATCH_LIMIT
    assert "static scratch" in toma.toma_status_str(SCRATCH_LIMIT)
