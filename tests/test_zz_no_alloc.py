"""The allocation-free column-sum entry point (collected last on purpose).

Some users of the library cannot allocate device memory where they call it (all device memory
was handed out at start-up, or the calling thread is not allowed the synchronisation an
allocation implies), so they cannot supply the scratch buffer bt_op_colsum asks for.
bt_op_colsum_static keeps its partial sums in an array built into the library instead.  It must
give the same result as the scratch-taking entry point, on the first call of a process and on
later calls that reuse the shared array with other sizes.
"""
import numpy as np
import pytest
import torch

import seeded_inputs as si
from paper_2606_24780_b200 import binding as b

from gpu_util import dev, empty, host, rel_l2, scratch

pytestmark = pytest.mark.gpu


def _reference(x, N, C):
    out = empty(C)
    nb = b.bt_op_colsum_scratch_bytes(N, C)
    b.bt_op_colsum(x, N, C, out, scratch(nb), nb)
    return out


def test_static_scratch_colsum_matches_scratch_entry_point_twice():
    # two calls in a row with different shapes: the second reuses (and must fully overwrite) the
    # part of the built-in array the first one used
    for seed, (N, C) in enumerate([(8192, 768), (1000, 3072)]):
        x = dev(si.normal_f32(90 + seed, (N, C), 1e-2))
        out = empty(C)
        # the allocator's count of allocation requests only ever grows (a garbage-collection pass
        # that frees older tensors during the call does not change it)
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        b.bt_op_colsum_static(x, N, C, out)
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before   # nothing allocated through torch either
        ref = _reference(x, N, C)
        assert torch.equal(out, ref)                           # same kernels, same order: same bits
        assert rel_l2(host(out), host(x).sum(0)) < 1e-5
        # torch's counter cannot see an allocation made inside the library; the driver's count of
        # free device bytes can.  From the second call on (the first one on a device may load the
        # library's module) a call must leave it exactly where it was.
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        b.bt_op_colsum_static(x, N, C, out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(out, ref)
    # a repeat of the first shape after the second
    x = dev(si.normal_f32(99, (8192, 768), 1e-2))
    out = empty(768)
    b.bt_op_colsum_static(x, 8192, 768, out)
    assert torch.equal(out, _reference(x, 8192, 768))


def test_static_scratch_colsum_rejects_oversized_and_bad_arguments():
    assert b.bt_op_colsum_static_max_floats() == 96 * 1024
    x = empty(64, 131072)            # one strip x 131072 floats of partial sums: over the limit
    assert b.bt_op_colsum_scratch_bytes(64, 131072) > 4 * b.bt_op_colsum_static_max_floats()
    with pytest.raises(b.BtError) as e:
        b.bt_op_colsum_static(x, 64, 131072, empty(131072))
    assert e.value.status == 2 and "scratch" in str(e.value)
    # the edge itself: 98,304 columns is the largest accepted width, the next multiple of four is refused
    edge = b.bt_op_colsum_static_max_floats()
    xe = dev(si.normal_f32(97, (64, edge), 1e-2))
    oute = empty(edge)
    b.bt_op_colsum_static(xe, 64, edge, oute)
    assert torch.equal(oute, _reference(xe, 64, edge))
    with pytest.raises(b.BtError) as e:
        b.bt_op_colsum_static(empty(64, edge + 4), 64, edge + 4, empty(edge + 4))
    assert e.value.status == 2
    with pytest.raises(b.BtError) as e:
        b.bt_op_colsum_static(x, 64, 6, empty(8))
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_op_colsum_static(None, 64, 768, empty(768))
    assert e.value.status == 1
