"""mfet_dedup_rows_static: dedup for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option: inside a serving
process whose GPU memory was all handed to another allocator at start-up, or on a
request thread that must never trigger the device-wide synchronisation that
cudaMalloc/cudaFree imply. For them the library carries a small fixed scratch array
of its own. This test calls that entry point through the C-ABI twice in a row (the
second call reuses the array with the first call's leftovers in it) and requires the
very same bits as mfet_dedup_rows, which sorts in a caller-provided workspace, and as
the CPU checker's sorted-unique definition (so the two GPU entry points cannot drift
together unnoticed). The file name makes pytest collect it after every other test.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from tests.helpers import mfet

pytestmark = pytest.mark.gpu


def _reference(m, rows_dev, n, max_row):
    """The existing entry point on a caller-allocated workspace."""
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        cap = n + 16
        ws = torch.empty(m.mfet_workspace_bytes(h, cap), dtype=torch.uint8, device="cuda")
        m.mfet_set_workspace(h, ws, ws.numel(), cap)
        uniq = torch.full((max(n, 1),), -1, dtype=torch.int64, device="cuda")
        inv = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
        nu = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        m.mfet_dedup_rows(h, rows_dev, n, uniq, inv, nu, max_row, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        k = int(nu.item())
        return k, uniq[:k].cpu().numpy(), inv[:n].cpu().numpy()
    finally:
        m.mfet_tables_destroy(h)


def test_static_dedup_matches_workspace_dedup_on_two_calls_in_a_row():
    m = mfet()
    rng = np.random.default_rng(2024)
    stream = torch.cuda.current_stream().cuda_stream
    dev = torch.cuda.current_device()
    # first a full-size call, then a smaller one over other values: leftovers of call 1 stay in the array
    cases = [(m.STATIC_DEDUP_MAX_IDS, 10**9, 10**9), (50_001, 30_000, 0), (0, 10, 0), (1, 5, 5)]
    for n, hi, max_row in cases:
        rows = torch.from_numpy(rng.integers(0, hi, size=n, dtype=np.int64)).cuda()
        if n == 0:
            rows = torch.zeros(1, dtype=torch.int64, device="cuda")
        uniq = torch.full((max(n, 1),), -1, dtype=torch.int64, device="cuda")
        inv = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
        nu = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        m.mfet_dedup_rows_static(dev, rows, n, uniq, inv, nu, max_row, stream)
        torch.cuda.synchronize()
        k = int(nu.item())
        k_ref, uniq_ref, inv_ref = _reference(m, rows, n, max_row)
        assert k == k_ref
        assert np.array_equal(uniq[:k].cpu().numpy(), uniq_ref)  # integer work: bit-exact
        assert np.array_equal(inv[:n].cpu().numpy(), inv_ref)
        want_uniq, want_inv = orc.dedup(rows[:n].cpu().numpy())
        assert k == want_uniq.size
        assert np.array_equal(uniq_ref, want_uniq)
        assert np.array_equal(inv_ref, want_inv)


def test_static_dedup_rejects_sizes_beyond_its_array():
    m = mfet()
    x = torch.zeros(8, dtype=torch.int64, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(m.MfetError) as e:
        m.mfet_dedup_rows_static(torch.cuda.current_device(), x, m.STATIC_DEDUP_MAX_IDS + 1, x, i, x)
    assert e.value.status == m.ERR_WORKSPACE
    with pytest.raises(m.MfetError) as e:
        m.mfet_dedup_rows_static(torch.cuda.current_device(), x, -1, x, i, x)
    assert e.value.status == m.ERR_INVALID_ARG
    with pytest.raises(m.MfetError) as e:
        m.mfet_dedup_rows_static(99, x, 4, x, i, x)
    assert e.value.status == m.ERR_INVALID_ARG
