"""Error paths that need a device but fault nothing: the host-side deadline of dd_sync (DD_ERR_TIMEOUT), a
bounded device-side wait that runs out (DD_ERR_WAIT_EXPIRED), and the error word read without synchronising.
No test here provokes a GPU fault, trap or hang: the only wait that runs out is limited to a few milliseconds
and every copy involved completes normally."""
import numpy as np
import pytest
import torch

from oracle import dd_oracle as orc
from tests._util import raw16

pytestmark = pytest.mark.gpu

HKV, D, T = 8, 128, 16


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


def _store_and_sets(B, P, k, seed=0):
    g = torch.Generator().manual_seed(seed)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()
    idx = torch.stack([torch.stack([torch.randperm(P, generator=g)[:k].sort().values for _ in range(HKV)])
                       for _ in range(B)]).to(torch.int32)
    return kv, idx


def test_sync_deadline_gives_timeout_then_succeeds(dd):
    """A few gathers of 64 MiB each are in flight (more than a millisecond apiece on the host link): a zero
    deadline reports DD_ERR_TIMEOUT without waiting, a generous one returns DD_OK, and nothing was lost."""
    B, P, k = 8, 256, 128
    kv, idx = _store_and_sets(B, P, k)
    copy = torch.cuda.Stream()
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, copy_stream=copy)
    idx_d = idx.cuda()
    torch.cuda.synchronize()
    for i in range(6):
        c.gather_kv_from_host(kv, idx_d, None, i % 2, stream=copy)
    with pytest.raises(dd.DDError) as e:
        c.sync(0.0)
    assert e.value.code == dd.DD_ERR_TIMEOUT and "busy" in str(e.value)
    c.sync(30.0)
    assert c.device_error() == (0, 0)
    assert np.array_equal(raw16(c.slot_tensor(1)), orc.gather_kv(raw16(kv), idx.numpy()))
    c.close()


def test_bounded_device_wait_runs_out_and_is_reported(dd):
    """The bulk gather's waits are bounded. With the test hook the first stage of block 0 expects 16 bytes more
    than its copy delivers, so that one wait cannot complete: after the limit (5 ms here) the block gives up,
    waits for its other copies in flight, returns, and the error word says DD_ERR_WAIT_EXPIRED. The context stays
    usable, and an ordinary gather on a fresh context is bit-exact."""
    B, P, k = 2, 96, 32
    kv, idx = _store_and_sets(B, P, k, seed=3)
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, gather_mode=dd.DD_GATHER_BULK, gather_ctas=4)
    with pytest.raises(dd.DDError):
        c.set_bulk_wait(0.0)
    c.set_bulk_wait(0.005, inflate_first_stage=True)
    c.gather_kv_from_host(kv, idx.cuda(), None, 0)
    c.sync(30.0)                                              # returns: nothing hangs
    assert c.last_device_error() == (dd.DD_ERR_WAIT_EXPIRED, 1)     # readable without synchronising
    assert c.device_error() == (dd.DD_ERR_WAIT_EXPIRED, 1)
    assert c.device_error() == (0, 0)
    # the same context without the hook: complete and bit-exact again
    c.set_bulk_wait(2.0, inflate_first_stage=False)
    c.gather_kv_from_host(kv, idx.cuda(), None, 1)
    assert c.device_error() == (0, 0)
    want = orc.gather_kv(raw16(kv), idx.numpy())
    assert np.array_equal(raw16(c.slot_tensor(1)), want)
    c.close()
    fresh = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, gather_mode=dd.DD_GATHER_BULK)
    fresh.gather_kv_from_host(kv, idx.cuda(), None, 0)
    assert fresh.device_error() == (0, 0)
    assert np.array_equal(raw16(fresh.slot_tensor(0)), want)
    fresh.close()
