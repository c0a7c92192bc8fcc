"""focus_count_kept_noalloc: the attended-pair count for callers that have no way to allocate
device memory (they were given buffers by someone else, or run where cudaMalloc is forbidden).
Its scratch is an array built into the library, so two things need checking that the workspace
variant never faces: the result must equal focus_count_kept's exactly, and a second call must not
be disturbed by what the first call left in the shared array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2604_03260_b200 import binding as fb
from paper_2604_03260_b200 import inputs as fi

pytestmark = pytest.mark.gpu


def masks_for(wl):
    shape = fb.shape_of(wl)
    Q, K, V, C = fi.make_inputs(wl, "cuda")
    mq = torch.empty((wl.Hq, wl.n), dtype=torch.int32, device="cuda")
    mk = torch.empty((wl.Hkv, wl.n), dtype=torch.int32, device="cuda")
    fb.focus_assign(shape, Q, wl.Hq, C, mq)
    fb.focus_assign(shape, K, wl.Hkv, C, mk)
    return shape, mq, mk


def with_workspace(shape, mq, mk):
    ws = fb.alloc_workspace(shape, 0)
    fb.focus_build_tiles(shape, mq, mk, 0, ws)
    out = torch.zeros(shape.batch * shape.Hq, dtype=torch.int64, device="cuda")
    fb.focus_count_kept(shape, mq, ws, out)
    torch.cuda.synchronize()
    return out.cpu()


def without_allocation(shape, mq, mk):
    out = torch.full((shape.batch * shape.Hq,), -7, dtype=torch.int64, device="cuda")   # must be overwritten
    fb.focus_count_kept_noalloc(shape, mq, mk, out)
    torch.cuda.synchronize()
    return out.cpu()


def test_two_calls_in_a_row_match_the_workspace_variant():
    # first call: a larger problem fills a long stretch of the built-in array ...
    big = fi.Workload("big", 8, 4, 128, 9000, 8, 2, 300, seed=77)
    shape, mq, mk = masks_for(big)
    assert torch.equal(without_allocation(shape, mq, mk), with_workspace(shape, mq, mk))
    # ... second call: a smaller, ragged problem with other masks reuses the same array
    small = fi.Workload("small", 4, 2, 64, 1000 + 37, 4, 1, 5, seed=78)
    shape2, mq2, mk2 = masks_for(small)
    got = without_allocation(shape2, mq2, mk2)
    assert torch.equal(got, with_workspace(shape2, mq2, mk2))
    assert (got > 0).all()
    # the count is the size of the attended set as the CPU oracle counts it from the mask definition
    want = fo.kept_pairs(mq2.cpu().numpy().view(np.uint32), mk2.cpu().numpy().view(np.uint32), small.window)
    assert np.array_equal(got.numpy(), want)
    # and the first problem again gives the first answer again
    assert torch.equal(without_allocation(shape, mq, mk), with_workspace(shape, mq, mk))


def test_sizes_beyond_the_builtin_array_are_refused():
    # 8 KV heads x 8192 key tiles x 4 groups x 16 B = 4 MiB > 1 MiB: refused before anything is launched
    shape = fb.make_shape(32, 8, 1 << 20, 128, 4, 2, 2048)
    dummy = torch.zeros(64, dtype=torch.int64, device="cuda")
    with pytest.raises(fb.FocusError) as e:
        fb.focus_count_kept_noalloc(shape, dummy, dummy, dummy)
    assert e.value.status == -3 and "1048576" in str(e.value)
    torch.cuda.synchronize()
