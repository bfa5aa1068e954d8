"""The allocation-free update entry point against the ordinary one.

`evk_q_update_static` exists for callers that cannot allocate device memory while they
run (a server whose memory was partitioned at start-up, a plug-in inside another
framework's budget): its scratch is a fixed array inside the library.  It must store
exactly the bits `evk_q_update` stores.  Two calls in a row are checked because the
scratch is shared and keeps what the previous call left in it.  This file sorts last
so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2603_10846_b200 import synth

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _twin_banks(evk, n, q0):
    bank = synth.gaussian_unit(n, 64, 123, DEV)
    mems = []
    for _ in range(2):
        mem = evk.evk_mem_create(64, n)
        evk.evk_mem_insert(mem, bank)
        for s in range(2):
            evk.evk_q_write(mem, s, torch.from_numpy(q0[s]).to(DEV))
        mems.append(mem)
    return mems


def test_static_scratch_update_matches_workspace_update_twice_in_a_row():
    from paper_2603_10846_b200 import evk
    n = 300000
    rng = np.random.default_rng(2024)
    q0 = rng.random((2, n)).astype(np.float32)
    ordinary, static = _twin_banks(evk, n, q0)
    # Batches above 8,192 updates take the multi-kernel sort, the path whose scratch is the fixed
    # array.  First a full-size batch with a very hot id, then ever shorter ones: keys, rewards or
    # histogram counts left behind beyond the new length would change the result.  The last two
    # are short enough for the single-kernel path, which needs no scratch at all.
    sizes = [65536, 20000, 9000, 65536, 8193, 5000, 777]
    batches = []
    for j, m in enumerate(sizes):
        hot = np.where(rng.random(m) < 0.2, 4242 + j, rng.integers(0, n if j % 2 == 0 else 3000, m))
        batches.append((hot.astype(np.int32), rng.standard_normal(m).astype(np.float32), j % 2, (0.05, 0.3, 1.0)[j % 3]))
    staged = [(torch.from_numpy(i).to(DEV), torch.from_numpy(r).to(DEV)) for i, r, _, _ in batches]
    torch.cuda.synchronize()
    for j, ((ids, r, stage, alpha), (ids_t, r_t)) in enumerate(zip(batches, staged)):
        evk.evk_q_update(ordinary, ids_t, stage, r_t, alpha)
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        evk.evk_q_update_static(static, ids_t, stage, r_t, alpha)
        torch.cuda.synchronize()
        if j > 0:      # (the first call on a device may load the module's code)
            assert torch.cuda.memory_allocated() == held            # nothing taken from torch's pool
            assert torch.cuda.mem_get_info()[0] == free             # nothing taken from the device
        for s in range(2):
            a = evk.evk_q_read(ordinary, s).cpu().numpy()
            b = evk.evk_q_read(static, s).cpu().numpy()
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32))     # bit-exact, as for evk_q_update
        assert evk.evk_last_status(static) == 0 and evk.evk_last_status(ordinary) == 0
    assert not np.array_equal(evk.evk_q_read(static, 0).cpu().numpy(), q0[0])  # something was written


def test_static_scratch_update_limits_and_rejections():
    from paper_2603_10846_b200 import evk
    n = 1000
    q0 = np.random.default_rng(7).random((2, n)).astype(np.float32)
    _, mem = _twin_banks(evk, n, q0)
    too_many = evk.EVK_Q_UPDATE_STATIC_MAX + 1
    with pytest.raises(evk.EvkError) as e:
        evk.evk_q_update_static(mem, torch.zeros(too_many, dtype=torch.int32, device=DEV), 0,
                                torch.zeros(too_many, device=DEV), 0.5)
    assert e.value.status == evk.EVK_ERR_UNSUPPORTED
    # a rejected batch (id out of range) writes nothing, and the next call works
    evk.evk_q_update_static(mem, torch.tensor([1, n, 2], dtype=torch.int32, device=DEV), 0,
                            torch.ones(3, device=DEV), 0.5)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q0[0].view(np.uint32))
    evk.evk_q_update_static(mem, torch.tensor([1, 1], dtype=torch.int32, device=DEV), 0,
                            torch.ones(2, device=DEV), 0.5)
    assert evk.evk_last_status(mem) == 0
    got = evk.evk_q_read(mem, 0).cpu().numpy()
    want = q0[0].copy()
    for _ in range(2):
        want[1] = np.float32(want[1] + np.float32(np.float32(0.5) * np.float32(np.float32(1.0) - want[1])))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the same on the multi-kernel path: a rejected long batch leaves its flag in the fixed array;
    # the next long batch must start from a clean one
    m = 12000
    rng = np.random.default_rng(8)
    ids = rng.integers(0, n, m).astype(np.int32)
    r = rng.random(m).astype(np.float32)
    bad_r = r.copy()
    bad_r[m // 2] = np.nan
    evk.evk_q_update_static(mem, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(bad_r).to(DEV), 0.5)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_NONFINITE
    assert np.array_equal(evk.evk_q_read(mem, 1).cpu().numpy().view(np.uint32), q0[1].view(np.uint32))
    twin, _ = _twin_banks(evk, n, q0)
    evk.evk_q_update(twin, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(r).to(DEV), 0.5)
    evk.evk_q_update_static(mem, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(r).to(DEV), 0.5)
    assert evk.evk_last_status(mem) == 0
    assert np.array_equal(evk.evk_q_read(mem, 1).cpu().numpy().view(np.uint32),
                          evk.evk_q_read(twin, 1).cpu().numpy().view(np.uint32))
