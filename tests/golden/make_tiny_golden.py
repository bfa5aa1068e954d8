"""Writes tests/golden/tiny_oracle.json: what the CPU oracle returns for the tiny workload
(N = 1,024, d = 768, fp32 embeddings rounded to bf16, 16 queries, k1 = 32, k2 = 4, w = 0.5, then
64 updates with alpha = 0.1), on inputs drawn by the seeded CPU generators.  Calls only the
oracle and the input generators.  Run from the repository root:

    python tests/golden/make_tiny_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2603_10846_b200 import synth  # noqa: E402


def compute():
    wl = synth.WORKLOADS["tiny"]
    bank = oracle.bf16_round(synth.make_bank(wl, "cpu").numpy())
    queries = oracle.bf16_round(synth.make_queries(wl, wl.batches[0], "cpu").numpy())
    q_tab = synth.make_q_tables(wl)
    out = {"citation": "Section 3.2 (two-phase retrieval) and Eq. 4 (value update) on the tiny synthetic bank; "
                       "values written by the CPU oracle, not taken from the paper",
           "checksum_bank": int(bank.astype(np.uint64).sum()), "checksum_queries": int(queries.astype(np.uint64).sum())}
    for stage in (0, 1):
        ids, scores, pool_ids, pool_sims = oracle.retrieve(bank, queries, q_tab[stage], wl.k1, wl.k2, wl.w)
        out[f"stage{stage}"] = {"ids": ids.tolist(), "pool_ids": pool_ids.tolist(),
                                "scores_hex": [[float(x).hex() for x in row] for row in scores]}
    u_ids, u_r = synth.make_updates(wl)
    q_after = oracle.q_update_f32(q_tab[0], u_ids, u_r, wl.alpha)
    out["update"] = {"ids": u_ids.tolist(), "rewards": u_r.tolist(),
                     "q_after_bits": q_after.view(np.uint32)[np.unique(u_ids)].tolist()}
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle.json")
    with open(path, "w") as f:
        json.dump(compute(), f)
    print("wrote", path)
