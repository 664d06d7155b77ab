"""The allocation-free statistics entry point against the regular request path.

Some hosts of this library may not call the CUDA allocator at all (their device memory is
pre-partitioned, or a cudaMalloc's implicit synchronisation is unacceptable where they run);
``bsa_mask_stats_noalloc`` serves them from a fixed scratch array inside the library.  Its numbers
must equal what ``bsa_plan_create`` reports for the same mask -- also on a second call, when the
shared scratch still holds the first call's contents.  Collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_25869_b200 import bsa
from paper_2609_25869_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _reference(mask_np, B_Q, B_KV, N, d):
    """Statistics through the existing entry point (plan creation)."""
    H = mask_np.shape[0]
    with bsa.plan_create(torch.from_numpy(mask_np).cuda(), B_Q, B_KV, N, H, d) as plan:
        inf = plan.info()
    return [inf["nnz_blocks"], inf["blocks_in_runs"], inf["max_row_nnz"]]


def test_no_alloc_stats_match_plan_create_on_two_calls_in_a_row():
    # two different masks, the larger first: stale counters or stale rows would show in the second
    big = I.config_mid().mask                                   # 8 x 128 x 128
    small = I.random_mask(17, 3, 40, 80, 0.3, empty_rows=0.25)  # 3 x 40 x 80, with empty rows
    out = torch.empty(4, dtype=torch.int64, device="cuda")
    for mask_np, (B_Q, B_KV, N, d) in ((big, (128, 128, 16384, 128)), (small, (64, 32, 40 * 64 - 7, 64))):
        got = bsa.mask_stats_noalloc(torch.from_numpy(mask_np).cuda(), out=out).cpu().tolist()
        assert got[:3] == _reference(mask_np, B_Q, B_KV, N, d)          # bit-exact: integer work
        assert got[3] == int((mask_np.sum(axis=2) == 0).sum())
    # the same mask twice in a row gives the same answer (accumulators are cleared per call)
    m = torch.from_numpy(small).cuda()
    a = bsa.mask_stats_noalloc(m).cpu().tolist()
    b = bsa.mask_stats_noalloc(m).cpu().tolist()
    assert a == b == got


def test_no_alloc_rejects_what_does_not_fit_or_is_malformed():
    L = bsa.lib()
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    m = torch.ones((1, 2, 2), dtype=torch.uint8, device="cuda")
    too_many = bsa.NOALLOC_MAX_ROWS + 1      # rows = heads * nQb; nothing is read before the size check
    assert L.bsa_mask_stats_noalloc(m.data_ptr(), 1, too_many, 1, out.data_ptr(), None) == 2
    assert L.bsa_mask_stats_noalloc(None, 1, 2, 2, out.data_ptr(), None) == 1
    assert L.bsa_mask_stats_noalloc(m.data_ptr(), 1, 2, 2, None, None) == 1
    assert L.bsa_mask_stats_noalloc(m.data_ptr(), 0, 2, 2, out.data_ptr(), None) == 1
    torch.cuda.synchronize()
    assert out.cpu().tolist() == [0, 0, 0, 0]      # rejected calls wrote nothing
    assert bsa.mask_stats_noalloc(m, out=out).cpu().tolist() == [4, 4, 2, 0]
