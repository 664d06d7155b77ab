"""The allocation-free statistics entry point, checked against the CPU oracle and the regular request path.

Some hosts of this library may not call the CUDA allocator at all (their device memory is
pre-partitioned, or a cudaMalloc's implicit synchronisation is unacceptable where they run);
``bsa_mask_stats_noalloc`` serves them from a fixed scratch array inside the library.  Its numbers
must equal the oracle's statistics of the same mask, and what ``bsa_plan_create`` reports -- also on
a second call, when the shared scratch still holds the first call's contents -- and a warm call
must leave the device's free memory where it was.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25869_b200 import bsa
from paper_2609_25869_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _plan_create_stats(mask_np, B_Q, B_KV, N, d):
    """Statistics through the existing entry point (plan creation)."""
    H = mask_np.shape[0]
    with bsa.plan_create(torch.from_numpy(mask_np).cuda(), B_Q, B_KV, N, H, d) as plan:
        inf = plan.info()
    return [inf["nnz_blocks"], inf["blocks_in_runs"], inf["max_row_nnz"]]


def _oracle_stats(mask_np):
    st = oracle.mask_stats(mask_np)
    return [st["nnz"], st["blocks_in_runs"], st["max_row_nnz"], int((mask_np.reshape(-1, mask_np.shape[2]).sum(axis=1) == 0).sum())]


def test_no_alloc_stats_match_the_oracle_and_plan_create_on_two_calls_in_a_row():
    # two different masks, the larger first: stale counters or stale rows would show in the second
    big = I.config_mid().mask                                   # 8 x 128 x 128
    small = I.random_mask(17, 3, 40, 80, 0.3, empty_rows=0.25)  # 3 x 40 x 80, with empty rows
    out = torch.empty(4, dtype=torch.int64, device="cuda")
    for mask_np, (B_Q, B_KV, N, d) in ((big, (128, 128, 16384, 128)), (small, (64, 32, 40 * 64 - 7, 64))):
        got = bsa.mask_stats_noalloc(torch.from_numpy(mask_np).cuda(), out=out).cpu().tolist()
        assert got == _oracle_stats(mask_np)                             # bit-exact: integer work
        assert got[:3] == _plan_create_stats(mask_np, B_Q, B_KV, N, d)
    # the same mask twice in a row gives the same answer (accumulators are cleared per call)
    m = torch.from_numpy(small).cuda()
    a = bsa.mask_stats_noalloc(m, out=out).cpu().tolist()
    b = bsa.mask_stats_noalloc(m, out=out).cpu().tolist()
    assert a == b == got


def test_no_alloc_warm_call_leaves_device_memory_untouched():
    """After the first call on the device (which resolves the scratch address and, with lazy module loading, lets the
    driver place the module), a call neither allocates nor frees: the driver's free-memory figure does not move."""
    m = torch.from_numpy(I.random_mask(3, 4, 64, 64, 0.5)).cuda()
    out = torch.empty(4, dtype=torch.int64, device="cuda")
    bsa.mask_stats_noalloc(m, out=out)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        bsa.mask_stats_noalloc(m, out=out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert out.cpu().tolist() == _oracle_stats(m.cpu().numpy())


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
