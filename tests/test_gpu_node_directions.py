"""Hash directions of every recursion node's own (variant of the causal recursion) on the GPU against the oracle:
bucket ids per level (bit for bit up to hash bits whose projection is next to zero), permutations from those ids,
outputs and row sums."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU

pytestmark = pytest.mark.gpu


def W(name, B, H, n, d, dtype, b, m, r, causal, n0, kind="gaussian", gen_seed=85, seed=0):
    return WL.Workload(name, B, H, n, d, dtype, b, m, r, causal, n0, kind, gen_seed, seed)


CASES = [
    W("nodedirs_two_levels", 1, 2, 2048, 64, "bf16", 128, 64, 6, True, 512, seed=1),
    W("nodedirs_four_levels_d128", 1, 2, 4096, 128, "bf16", 64, 48, 7, True, 256, seed=2),
    W("nodedirs_ragged_n3001", 1, 1, 3001, 64, "bf16", 96, 40, 6, True, 400, seed=3),
    W("nodedirs_fp32", 1, 1, 1024, 64, "fp32", 64, 32, 5, True, 128, seed=4),
    W("nodedirs_chunked_leaves", 1, 1, 12288, 64, "bf16", 256, 128, 7, True, 3072, seed=5),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_node_directions_match_the_oracle(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=True, n0=w.n0, seed=w.seed, out_dtype=torch.float32, debug=True,
                                 node_directions=True)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (WL.as_f64(x) for x in arrs)
    gq, gk = inter["q_ids"].cpu().numpy(), inter["k_ids"].cpu().numpy()          # [L, G, n]
    pq, pk, rk = (inter[x].cpu().numpy() for x in ("perm_q", "perm_k", "rank_k"))
    L, leaf = O.causal_grid(w.n, w.n0)
    assert gq.shape == (L, w.G, w.n)
    amb_total = mism_total = 0
    for g in range(w.G):
        for level in range(L):
            s = leaf << (L - 1 - level)
            for j in range(1 << level):
                q0, k0 = (2 * j + 1) * s, 2 * j * s
                nq = max(0, min(s, w.n - q0))
                if nq == 0 or w.b >= s:
                    continue
                node = O.heap_node(level, j)
                Wn = O.directions(w.d, w.r, w.seed, node=node)
                assert np.array_equal(Wn, ha.get_projections(w.d, w.r, w.seed, node=node))
                for X, got in ((Q64[g][q0:q0 + nq], gq[level, g, q0:q0 + nq]), (K64[g][k0:k0 + s], gk[level, g, k0:k0 + s])):
                    ids, absp = O.bucket_ids(X, Wn)
                    amb = absp < PU.AMBIGUOUS
                    amb_total += int(amb.sum())
                    for i in np.nonzero(ids != got)[0]:
                        mism_total += 1
                        diff = (int(ids[i]) ^ (int(ids[i]) >> 1)) ^ (int(got[i]) ^ (int(got[i]) >> 1))
                        assert all(amb[i, t] for t in range(w.r) if diff >> t & 1), (g, level, j, i)
                perm, _ = O.stable_argsort(gq[level, g, q0:q0 + nq])
                assert (pq[level, g, j * s:j * s + nq] == perm).all()
                perm, rank = O.stable_argsort(gk[level, g, k0:k0 + s])
                assert (pk[level, g, j * s:(j + 1) * s] == perm).all() and (rk[level, g, j * s:(j + 1) * s] == rank).all()
    PU.check_samples(w, inter)
    Wd = O.directions(w.d, w.r, w.seed)
    o_np, l_np = out.cpu().numpy().reshape(w.G, w.n, w.d), lse.cpu().numpy().reshape(w.G, w.n)
    errs, lerrs = [], []
    for g in range(w.G):
        ro, rl = O.segment_forward(Q64[g], K64[g], V64[g], Wd, w.b, w.m, True, w.n0, w.seed, g, scale=1.0 / math.sqrt(w.d),
                                   ids_q=gq[:, g], ids_k=gk[:, g], node_directions=True)
        errs.append(np.abs(o_np[g] - ro)); lerrs.append(np.abs(l_np[g] - rl) / np.maximum(np.abs(rl), 1.0))
    err, lerr = np.concatenate(errs), np.concatenate(lerrs)
    print(w.name, "ambiguous bits", amb_total, "id mismatches", mism_total, "max", err.max(), "mean", err.mean(), "lse", lerr.max())
    assert err.max() <= PU.OUT_MAX_ABS and err.mean() <= PU.OUT_MEAN_ABS and lerr.max() <= PU.LSE_REL
    # the variant changes the result below the root, and only there
    out0, _ = ha.forward(q, k, v, w.b, w.m, w.r, causal=True, n0=w.n0, seed=w.seed, out_dtype=torch.float32)
    assert not torch.equal(out0, out)
