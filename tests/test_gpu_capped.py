"""Alg. 2 with its caps (probe rows T, tau, the upper cap C_i and the lower cap tau / kappa) on the GPU against the
oracle: the probe positions bit for bit, tau within the logarithmic tolerance of the row sums, outputs and row sums
within the tolerances of the uncapped path; caps that never bind give the uncapped result."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU

pytestmark = pytest.mark.gpu


def W(name, B, H, n, d, b, m, r, causal, n0, kind="gaussian", gen_seed=70, seed=0, n_k=0):
    return WL.Workload(name, B, H, n, d, "bf16", b, m, r, causal, n0, kind, gen_seed, seed, n_k)


CASES = [
    (W("capped_d64", 1, 2, 2048, 64, 128, 96, 6, False, 0, seed=1), (4.0, 8.0)),
    (W("capped_d128_binding", 1, 2, 2048, 128, 256, 128, 7, False, 0, seed=2), (0.5, 100.0)),
    (W("capped_causal_three_levels", 1, 2, 4096, 64, 128, 64, 6, True, 512, seed=3), (2.0, 4.0)),
    (W("capped_causal_ragged_d128", 1, 1, 3001, 128, 96, 48, 6, True, 400, seed=4), (1.0, 16.0)),
    (W("capped_clustered", 1, 2, 4096, 64, 256, 256, 7, False, 0, kind="clustered", seed=5), (8.0, 2.0)),
    (W("capped_heavy_tail", 1, 2, 2048, 64, 128, 128, 7, False, 0, kind="student_t", seed=6), (8.0, 16.0)),
    (W("capped_cross_sides", 1, 2, 1500, 64, 128, 64, 6, False, 0, seed=7, n_k=2500), (2.0, 8.0)),
    (W("capped_lower_cap_everywhere", 1, 1, 1024, 64, 64, 16, 5, False, 0, seed=8), (1e-3, 1.5)),
]


def node_list(w):
    for level, s in PU.levels_of(w):
        for j in range((1 << level) if w.causal else 1):
            q0, k0, s_, nq = PU.node_ranges(w, level, j)
            if nq > 0 and w.b < s_:
                yield (O.heap_node(level, j) if w.causal else 0), q0, k0, s_, nq


@pytest.mark.parametrize("w,caps", CASES, ids=[w.name for w, _ in CASES])
def test_capped_forward_matches_the_oracle(w, caps):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, out_dtype=torch.float32,
                                 debug=True, caps=caps)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (WL.as_f64(x) for x in arrs)
    gq, gk = inter["q_ids"].cpu().numpy(), inter["k_ids"].cpu().numpy()
    tpos, ltau = inter["row_subset"].cpu().numpy(), inter["log2_tau"].cpu().numpy()
    scale = 1.0 / math.sqrt(w.d)
    for g in range(w.G):
        for node, q0, k0, s, nq in node_list(w):
            T = O.row_subset(w.seed, g, node, w.m, nq)
            assert (tpos[g, node, :w.m] == T).all(), (g, node)
            perm_q, rank_q = O.stable_argsort(gq[g, q0:q0 + nq])
            _, rank_k = O.stable_argsort(gk[g, k0:k0 + s])
            ref = O.unmasked_row_sum_bound(Q64[g][q0:q0 + nq], K64[g][k0:k0 + s], rank_q, rank_k, perm_q[T], w.b,
                                           O.query_block_size(nq, s, w.b), scale)
            got = ltau[g, node] * math.log(2.0)
            assert abs(got - ref) <= PU.LSE_REL * max(abs(ref), 1.0), (g, node, got, ref)
    # heavy values: the weights are single bf16 numbers here, so the derived bound 2^-8 max|v| (times the largest
    # ratio of uncapped to capped row sum, which the capped normalisation can reach) is what holds
    bound = None
    if PU.heavy_values(w):
        bound = float(np.abs(V64).max()) / 256.0
    # a capped row's output is its uncapped output times (uncapped row sum / capped row sum): errors are measured
    # in units of that factor (1 where the caps do not bind)
    out0, lse0 = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, out_dtype=torch.float32)
    ratio = np.maximum(1.0, np.exp((lse0 - lse).double().cpu().numpy())).reshape(w.G, w.n)
    stats = PU.check_outputs(w, Q64, K64, V64, out, lse, inter, caps=caps, max_abs_bound=bound, row_scale=ratio)
    # the caps must matter in the cases built for it
    print(w.name, stats, "largest change of lse by the caps", float((lse - lse0).abs().max()))
    if "binding" in w.name or "lower_cap" in w.name:
        assert float((lse - lse0).abs().max()) > 1e-2


def test_caps_that_never_bind_give_the_uncapped_result():
    w = CASES[0][0]
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    o0, l0 = ha.forward(q, k, v, w.b, w.m, w.r, seed=w.seed, out_dtype=torch.float32)
    o1, l1 = ha.forward(q, k, v, w.b, w.m, w.r, seed=w.seed, out_dtype=torch.float32, caps=(1e30, 1e30))
    torch.cuda.synchronize()
    # same weights and products; only the normaliser differs (the unrounded row sum instead of the sum of the
    # bf16-rounded weights): relative 2^-9 at most
    assert float((l1 - l0).abs().max()) <= 1e-5
    assert float((o1 - o0).abs().max()) <= 2.0 ** -8 * float(o0.abs().max())


def test_capped_arguments_are_checked():
    w = CASES[0][0]
    q, k, v = PU.to_device(w, WL.make_inputs(w))
    with pytest.raises(ha.HyperAttnError, match="invalid argument"):
        ha.forward(q, k, v, w.b, w.m, w.r, caps=(0.0, 2.0))
    with pytest.raises(ha.HyperAttnError, match="unsupported shape"):
        ha.forward(q, k, v, w.b, w.m, w.r, caps=(1.0, 2.0), precise=True)


def test_caps_reduce_the_spread_of_the_row_sums_on_heavy_tailed_inputs():
    """The benchmark's heavy-tailed kind (Student-t entries clipped at +-20, d = 128, b = 128, m = 512, r = 8) at
    4096 rows, 24 seeds (each seed redraws directions, samples and probe rows): variance over the seeds of
    ln d~_i, averaged over the rows, with and without the caps."""
    w = W("capped_variance", 1, 2, 4096, 128, 128, 512, 8, False, 0, kind="student_t", seed=0)
    q, k, v = PU.to_device(w, WL.make_inputs(w))
    un, cp = [], []
    for seed in range(24):
        un.append(ha.forward(q, k, v, w.b, w.m, w.r, seed=seed)[1].double().cpu().numpy())
        cp.append(ha.forward(q, k, v, w.b, w.m, w.r, seed=seed, caps=(8.0, 16.0))[1].double().cpu().numpy())
    var_un, var_cp = float(np.var(np.array(un), axis=0).mean()), float(np.var(np.array(cp), axis=0).mean())
    print("variance of ln d~ over seeds, mean over rows: uncapped", var_un, "capped", var_cp)
    assert var_cp < var_un
