"""Host-buffer calls with a page-locked staging buffer (evk_mem_set_host_staging): updates and
inserts return without waiting for the device, retrieval results are written into the staging
buffer by the merge kernel.  Results must be those of the calls without staging, and the
caller's arrays must be free for reuse the moment a call returns."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth
from tests.test_gpu_parity import DEV, make_mem, run_retrieve

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def evk():
    from paper_2603_10846_b200 import evk as _evk
    return _evk


def _bank(evk, n=30000, d=256, seed=700):
    bank = synth.gaussian_unit(n, d, seed, DEV)
    q_tab = np.random.default_rng(seed + 1).random((2, n)).astype(np.float32)
    return bank, q_tab, make_mem(evk, bank, q_tab)


def test_staged_retrieve_equals_the_device_call(evk):
    bank, q_tab, mem = _bank(evk)
    evk.evk_mem_set_host_staging(mem, 1 << 20)
    for b, k1, k2 in ((1, 16, 1), (8, 64, 8), (300, 128, 32)):
        queries = synth.gaussian_unit(b, bank.shape[1], 710 + b, DEV)
        want = run_retrieve(evk, mem, queries, 1, k1, k2, 0.5)
        ids_h = torch.full((b, k2), -9, dtype=torch.int32)           # pageable on purpose
        sc_h = torch.full((b, k2), -9.0, dtype=torch.float32)
        evk.evk_retrieve_host(mem, queries.cpu(), 1, k1, k2, 0.5, ids_h, sc_h)
        assert np.array_equal(ids_h.numpy(), want[0]) and np.array_equal(sc_h.numpy(), want[1])


def test_staged_updates_leave_the_callers_arrays_free(evk):
    # nine batches back to back (more than the four slots), each overwritten the moment the call
    # returns; no synchronise in between: the table must equal the oracle's, bit for bit
    bank, q_tab, mem = _bank(evk, n=20000, d=64)
    evk.evk_mem_set_host_staging(mem, 4 << 20)
    rng = np.random.default_rng(720)
    ids_h = torch.empty(70000, dtype=torch.int32).pin_memory()
    r_h = torch.empty(70000, dtype=torch.float32).pin_memory()
    q_orc = q_tab[0].copy()
    for m in (5, 1024, 3000, 65536, 70000, 17, 2048, 9000, 64):    # 70,000 ids do not fit a slot: path without staging
        ids = np.where(rng.random(m) < 0.2, 77, rng.integers(0, 20000, m)).astype(np.int32)
        r = rng.standard_normal(m).astype(np.float32)
        ids_h[:m] = torch.from_numpy(ids)
        r_h[:m] = torch.from_numpy(r)
        evk.evk_q_update_host(mem, ids_h[:m], 0, r_h[:m], 0.3)
        ids_h.fill_(-1)            # an id the device would reject, were it still reading these arrays
        r_h.fill_(float("nan"))
        q_orc = oracle.q_update_f32(q_orc, ids, r, 0.3)
    torch.cuda.synchronize()
    assert evk.evk_last_status(mem) == 0
    assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q_orc.view(np.uint32))


def test_staged_inserts_and_a_retrieval_that_finds_them(evk):
    n0, d = 5000, 128
    bank = synth.gaussian_unit(n0, d, 730, DEV)
    mem = evk.evk_mem_create(d, n0 + 4000, 2, q_default=0.25)
    evk.evk_mem_insert(mem, bank, evk.EVK_STAGE_ALL)
    evk.evk_mem_set_host_staging(mem, 256 << 10)                    # 64 KB slots: 256 bf16 rows fit, 600 do not
    rows_h = torch.empty((600, d), dtype=torch.bfloat16).pin_memory()
    q0_h = torch.empty(600, dtype=torch.float32).pin_memory()
    added, q_added = [], []
    for j, n_new in enumerate((16, 1, 200, 600, 3)):
        rows = synth.gaussian_unit(n_new, d, 740 + j, "cpu")
        q0 = torch.from_numpy(np.random.default_rng(750 + j).random(n_new).astype(np.float32))
        rows_h[:n_new] = rows
        q0_h[:n_new] = q0
        evk.evk_mem_insert_host(mem, rows_h[:n_new], 1, q0_h[:n_new])
        rows_h.zero_()
        q0_h.fill_(-5.0)
        added.append(rows)
        q_added.append(q0)
    added, q_added = torch.cat(added), torch.cat(q_added)
    assert evk.evk_mem_size(mem) == n0 + added.shape[0]
    got = evk.evk_bank_read(mem, n0, added.shape[0]).cpu()
    assert torch.equal(got.view(torch.int16), added.view(torch.int16))
    assert torch.equal(evk.evk_q_read(mem, 1).cpu()[n0:], q_added)
    assert torch.all(evk.evk_q_read(mem, 0).cpu()[n0:] == 0.25)      # the stage the insert did not name
    # each new row is its own nearest neighbour
    pick = torch.arange(0, added.shape[0], 37)
    ids_h = torch.empty((pick.numel(), 1), dtype=torch.int32)
    sc_h = torch.empty((pick.numel(), 1), dtype=torch.float32)
    evk.evk_retrieve_host(mem, added[pick].contiguous(), 1, 8, 1, 0.0, ids_h, sc_h)   # w = 0: similarity alone
    assert torch.equal(ids_h[:, 0].long(), pick + n0)


def test_device_findings_of_a_staged_update_reach_the_status_word(evk):
    bank, q_tab, mem = _bank(evk, n=4000, d=64)
    evk.evk_mem_set_host_staging(mem, 64 << 10)
    bad = torch.tensor([1, 4000 + 5, 2], dtype=torch.int32)
    evk.evk_q_update_host(mem, bad, 0, torch.ones(3), 0.5)            # returns at once, no exception
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q_tab[0].view(np.uint32))


def test_staging_buffer_is_checked_and_can_be_withdrawn(evk):
    bank, q_tab, mem = _bank(evk, n=4000, d=64)
    lib = evk._lib
    pageable = torch.empty(1 << 20, dtype=torch.uint8)
    ptr = pageable.data_ptr() + (-pageable.data_ptr()) % 256
    assert lib.evk_mem_set_host_staging(mem.handle, ctypes.c_void_p(ptr), 1 << 19) == evk.EVK_ERR_INVALID
    pinned = torch.empty((1 << 20) + 256, dtype=torch.uint8).pin_memory()
    p = pinned.data_ptr() + (-pinned.data_ptr()) % 256
    assert lib.evk_mem_set_host_staging(mem.handle, ctypes.c_void_p(p + 8), 1 << 19) == evk.EVK_ERR_INVALID   # alignment
    assert lib.evk_mem_set_host_staging(mem.handle, ctypes.c_void_p(p), 8192) == evk.EVK_ERR_INVALID          # too small
    assert lib.evk_mem_set_host_staging(mem.handle, ctypes.c_void_p(bank.data_ptr()), 1 << 19) == evk.EVK_ERR_INVALID  # device memory
    assert lib.evk_mem_set_host_staging(mem.handle, ctypes.c_void_p(p), 1 << 20) == evk.EVK_OK
    ids = torch.arange(100, dtype=torch.int32)
    evk.evk_q_update_host(mem, ids, 0, torch.ones(100), 1.0)
    assert lib.evk_mem_set_host_staging(mem.handle, None, 0) == evk.EVK_OK      # waits for the update, then lets go
    pinned.fill_(0xff)
    evk.evk_q_update_host(mem, ids + 100, 0, torch.ones(100), 1.0)               # synchronising path again
    q = evk.evk_q_read(mem, 0).cpu().numpy()
    assert np.all(q[:200] == 1.0) and np.array_equal(q[200:], q_tab[0][200:])
