"""Seeded random shapes, modes and tie patterns through the retrieval and the update, each judged
against the CPU oracle: a net for the corners the hand-picked cases leave between them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def evk():
    from paper_2603_10846_b200 import evk as _evk
    return _evk


@pytest.mark.parametrize("seed", range(6))
def test_random_retrievals(evk, seed):
    rng = np.random.default_rng(1000 + seed)
    done = 0
    while done < 12:
        d = int(rng.choice([64, 72, 200, 256, 768, 776, 1024, 2048]))
        n = int(rng.choice([1, 7, 255, 257, 4097, 16385, 50000, 150000]))
        n = min(n, 150000 * 1024 // d)
        b = int(rng.choice([1, 3, 9, 17, 63, 64, 65, 129, 257, 300]))
        k1 = int(rng.choice([1, 5, 31, 64, 100, 256, 257, 512]))
        k2 = int(rng.integers(1, min(k1, 40) + 1)) if rng.random() < 0.8 else k1
        w = float(rng.choice([0.0, 0.25, 0.5, 1.0]))
        mode = int(rng.choice([evk.EVK_SCORING_AUTO, evk.EVK_SCORING_TENSOR, evk.EVK_SCORING_STREAM]))
        zscore = bool(rng.random() < 0.25)
        case_seed = int(rng.integers(1 << 30))
        bank = synth.gaussian_unit(n, d, case_seed, DEV).to(torch.bfloat16)
        if rng.random() < 0.25 and n > 4:
            bank[n // 2:] = bank[: n - n // 2].clone()            # duplicated rows: exact similarity ties
        queries = synth.gaussian_unit(b, d, case_seed + 1, DEV).to(torch.bfloat16)
        q_tab = np.random.default_rng(case_seed).random((2, n)).astype(np.float32)
        if rng.random() < 0.25:
            q_tab = (np.round(q_tab * 4) / 4).astype(np.float32)  # ties in the values as well
        mem = evk.evk_mem_create(d, n)
        evk.evk_mem_set_scoring(mem, mode)
        evk.evk_mem_set_score_norm(mem, evk.EVK_NORM_POOL_ZSCORE if zscore else evk.EVK_NORM_NONE)
        evk.evk_mem_insert(mem, bank)
        for s in range(2):
            evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(DEV))
        try:
            out = evk.evk_retrieve(mem, queries, 1, k1, k2, w, return_pool=True)
        except evk.EvkError as e:
            assert e.status == evk.EVK_ERR_UNSUPPORTED and mode == evk.EVK_SCORING_TENSOR
            continue
        torch.cuda.synchronize()
        case = dict(n=n, d=d, b=b, k1=k1, k2=k2, w=w, mode=mode, zscore=zscore, seed=case_seed)
        assert evk.evk_last_status(mem) == 0, case
        out = [x.cpu().numpy() for x in out]
        sample = list(range(b)) if b <= 4 else sorted(rng.choice(b, 4, replace=False).tolist())
        try:
            parity.check_retrieve(synth.bf16_bits(bank), synth.bf16_bits(queries), q_tab[1], k1, k2, w, out,
                                  sample=sample, zscore=zscore)
        except AssertionError as e:
            raise AssertionError(f"{case}: {e}") from e
        done += 1


@pytest.mark.parametrize("seed", range(3))
def test_random_updates(evk, seed):
    rng = np.random.default_rng(2000 + seed)
    for _ in range(12):
        n = int(rng.choice([1, 5, 300, 70000, (1 << 20) + 3]))
        m = int(rng.choice([0, 1, 63, 1024, 2048, 2049, 4000, 8192, 8193, 20000, 65536, 65537, 100000]))
        alpha = float(rng.choice([1.0, 0.5, 0.1, 0.05]))
        kind = str(rng.choice(["uniform", "hot", "zipf"]))
        if kind == "uniform":
            ids = rng.integers(0, n, m)
        elif kind == "hot":
            ids = np.where(rng.random(m) < 0.5, rng.integers(0, n), rng.integers(0, n, m))
        else:
            ids = np.minimum(rng.zipf(1.1, m) - 1, n - 1)
        ids = ids.astype(np.int32)
        rewards = rng.lognormal(0, 0.5, m).astype(np.float32)
        q0 = rng.random(n).astype(np.float32)
        which = str(rng.choice(["plain", "static", "decay"]))
        if which == "static" and m > 65536:
            which = "plain"
        mem = evk.evk_mem_create(64, n)
        evk.evk_mem_insert(mem, torch.zeros((n, 64), device=DEV, dtype=torch.bfloat16))
        evk.evk_q_write(mem, 1, torch.from_numpy(q0).to(DEV))
        t_ids, t_r = torch.from_numpy(ids).to(DEV), torch.from_numpy(rewards).to(DEV)
        if which == "plain":
            evk.evk_q_update(mem, t_ids, 1, t_r, alpha)
        elif which == "static":
            evk.evk_q_update_static(mem, t_ids, 1, t_r, alpha)
        else:
            evk.evk_q_update_decay(mem, t_ids, 1, t_r)
        torch.cuda.synchronize()
        case = dict(n=n, m=m, alpha=alpha, kind=kind, which=which)
        assert evk.evk_last_status(mem) == 0, case
        got = evk.evk_q_read(mem, 1).cpu().numpy()
        if which == "decay":
            want, _ = oracle.q_update_decay(q0, np.zeros(n, np.uint32), ids, rewards)
            assert np.array_equal(want.view(np.uint32), got.view(np.uint32)), case
        else:
            parity.check_update(q0, ids, rewards, alpha, got)
