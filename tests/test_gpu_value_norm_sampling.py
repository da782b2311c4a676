"""Residual columns drawn by squared row norms of V (Lemma 2) on the GPU against the oracle: the drawn indices bit
for bit (the distribution is made of integers on both sides), their weights, and the outputs and row sums."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU
from test_gpu_capped import node_list

pytestmark = pytest.mark.gpu


def W(name, B, H, n, d, b, m, r, causal, n0, kind="gaussian", gen_seed=80, seed=0, n_k=0):
    return WL.Workload(name, B, H, n, d, "bf16", b, m, r, causal, n0, kind, gen_seed, seed, n_k)


CASES = [
    W("vnorm_d64", 1, 2, 2048, 64, 128, 96, 6, False, 0, seed=1),
    W("vnorm_d128", 1, 2, 2048, 128, 256, 128, 7, False, 0, seed=2),
    W("vnorm_causal_three_levels", 1, 2, 4096, 64, 128, 64, 6, True, 512, seed=3),
    W("vnorm_causal_ragged_d128", 1, 1, 3001, 128, 96, 48, 6, True, 400, seed=4),
    W("vnorm_heavy_tail", 1, 2, 2048, 64, 128, 128, 7, False, 0, kind="student_t", seed=5),
    W("vnorm_cross_sides_max_samples", 1, 2, 1500, 64, 128, 512, 6, False, 0, seed=6, n_k=5000),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_value_norm_sampling_matches_the_oracle(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, out_dtype=torch.float32,
                                 debug=True, value_norm_sampling=True)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (WL.as_f64(x) for x in arrs)
    smp, wl = inter["samples"].cpu().numpy(), inter["sample_log2w"].cpu().numpy().astype(np.float64)
    for g in range(w.G):
        wq = O.value_norm_weights(V64[g])
        for node, q0, k0, s, nq in node_list(w):
            idx, sw = O.sample_by_value_norms(w.seed, g, node, w.m, wq[k0:k0 + s])
            assert (smp[g, node, :w.m] == idx).all(), (g, node)
            np.testing.assert_allclose(wl[g, node, :w.m], np.log2(sw), atol=1e-5)
    gq, gk = inter["q_ids"].cpu().numpy(), inter["k_ids"].cpu().numpy()
    errs, lerrs = [], []
    Wd = O.directions(w.d, w.r, w.seed)
    o_np, l_np = out.cpu().numpy().reshape(w.G, w.n, w.d), lse.cpu().numpy().reshape(w.G, w.n)
    for g in range(w.G):
        ro, rl = O.segment_forward(Q64[g], K64[g], V64[g], Wd, w.b, w.m, w.causal, w.n0, w.seed, g, scale=1.0 / math.sqrt(w.d),
                                   ids_q=gq[g], ids_k=gk[g], value_norm_sampling=True)
        errs.append(np.abs(o_np[g] - ro)); lerrs.append(np.abs(l_np[g] - rl) / np.maximum(np.abs(rl), 1.0))
    err, lerr = np.concatenate(errs), np.concatenate(lerrs)
    bound = PU.OUT_MAX_ABS if not PU.heavy_values(w) else float(np.abs(V64).max()) / 256.0     # single bf16 weights: 2^-8 max|v|
    print(w.name, "max", err.max(), "mean", err.mean(), "lse", lerr.max(), "bound", bound)
    assert err.max() <= bound and err.mean() <= PU.OUT_MEAN_ABS and lerr.max() <= PU.LSE_REL


def test_value_norm_sampling_prefers_long_value_rows_and_checks_its_arguments():
    w = CASES[0]
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    v = v.clone()
    v[:, :, ::2] *= 0.05                                   # every other value row almost vanishes
    _, _, inter = ha.forward(q, k, v, w.b, w.m, w.r, seed=w.seed, debug=True, value_norm_sampling=True)
    smp = inter["samples"].cpu().numpy()[:, 0, :w.m]
    assert (smp % 2 == 1).mean() > 0.98
    with pytest.raises(ha.HyperAttnError, match="unsupported shape"):
        ha.forward(q, k, v, w.b, 600, w.r, value_norm_sampling=True)                 # more samples than the table of column weights holds
    with pytest.raises(ha.HyperAttnError, match="unsupported shape"):
        ha.forward(q, k, v, w.b, w.m, w.r, value_norm_sampling=True, precise=True)
