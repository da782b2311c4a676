"""Backward pass at the full benchmark sizes, in the launch configuration the benchmark times.

The dense fp64 backward of the oracle cannot hold these sizes, so the check uses what can be
computed row by row and what holds at any size:

* dQ of sampled query rows against central differences of the oracle's forward pass: with the
  bucket ids (hence the permutations) and the samples fixed, dQ_i is the gradient of
  f(q_i) = <dO_i, out_i(q_i)> in q_i, and out_i can be evaluated for one row;
* every row of P sums to one (the saved lse is the logarithm of the row's weighted sum), so
  sum_j dV_j = sum_i dO_i, and sum_j dS_ij = <dO_i, O_i> - delta_i = 0, so sum_j dK_j = 0;
* dV_j and dK_j of a few keys j element by element (the two smaller workloads): the oracle's forward pass, given
  one-hot "values" e_j, returns column j of P for every row, and dV_j = sum_i P_ij dO_i,
  dK_j = scale sum_i P_ij (<dO_i, v_j> - <dO_i, O_i>) q_i need nothing else.

Tolerances: P and dS are rounded to bf16 before the tensor-core products and O enters delta in
bf16, so, as in the small-size parity test, a dQ entry may be off by 2^-6 of the summed absolute
values of its terms, scale * sum_j P_ij (|dP_ij| + |delta_i| + sum_c |dO_ic O_ic|) |K_jc|; the
oracle's forward pass evaluates those P-weighted sums row by row when it is given |K| (times
|dP_i.|) in the place of V.  The column sums run over G*n fp32 reductions of bf16-rounded
terms: 2^-7 of the sum of absolute values."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU

pytestmark = pytest.mark.gpu

FULL = [WL.CONFIGS[1], WL.CONFIGS[2], WL.CONFIGS[3], WL.CONFIGS[4]]
SUM_REL = 2.0 ** -7
TERMS_REL = 2.0 ** -6


@pytest.mark.parametrize("w", FULL, ids=[w.name for w in FULL])
def test_backward_full_size_rows_and_sums(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, debug=True)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4242 + w.seed)
    dout = torch.randn((w.B, w.H, w.n, w.d), device="cuda", generator=gen, dtype=torch.float32).to(torch.bfloat16)
    dq, dk, dv = ha.backward(q, k, v, out, lse, dout, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed,
                             grad_dtype=torch.float32)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    for x in (dq, dk, dv):
        assert bool(torch.isfinite(x).all())

    # ---- column sums, every segment ---------------------------------------------------------
    do64 = dout.double().reshape(w.G, w.n, w.d)
    dv64, dk64 = dv.double().reshape(w.G, w.n, w.d), dk.double().reshape(w.G, w.n, w.d)
    sum_err = (dv64.sum(1) - do64.sum(1)).abs().max().item()
    sum_size = do64.abs().sum(1).max().item()
    assert sum_err <= SUM_REL * sum_size, ("sum dV", sum_err, sum_size)
    dk_err = dk64.sum(1).abs().max().item()
    dk_size = dk64.abs().sum(1).max().item()
    assert dk_err <= SUM_REL * dk_size, ("sum dK", dk_err, dk_size)

    # ---- dQ rows by central differences of the oracle's forward pass ------------------------
    g = w.G - 1
    Q64, K64, V64 = (WL.as_f64(x[g]) for x in arrs)
    ids_q, ids_k = inter["q_ids"][g].cpu().numpy(), inter["k_ids"][g].cpu().numpy()
    W = O.directions(w.d, w.r, w.seed)
    scale = 1.0 / math.sqrt(w.d)
    dO = do64[g].cpu().numpy()
    got = dq.double().reshape(w.G, w.n, w.d)[g].cpu().numpy()
    h = 1e-4
    worst = 0.0
    for i in (5, w.n // 2 - 1, w.n // 2, w.n // 2 + 131, w.n - 3):       # (the middle rows sit on the top split of Alg. 4)
        rows = np.array([i])

        def f(qrow):
            Qm = Q64.copy()
            Qm[i] = qrow
            o, _ = O.segment_forward(Qm, K64, V64, W, w.b, w.m, w.causal, w.n0, w.seed, g, scale=scale,
                                     rows=rows, ids_q=ids_q, ids_k=ids_k)
            return float(np.dot(o[0], dO[i]))

        want = np.zeros(w.d)
        for c in range(w.d):
            e = np.zeros(w.d)
            e[c] = h
            want[c] = (f(Q64[i] + e) - f(Q64[i] - e)) / (2 * h)
        # the summed absolute values of an entry's terms, as in the small-size parity test: the oracle's forward
        # pass, given other "values", returns sum_j P_ij x_j for any per-key vectors x_j
        def p_weighted(X):
            o, _ = O.segment_forward(Q64, K64, X, W, w.b, w.m, w.causal, w.n0, w.seed, g, scale=scale,
                                     rows=rows, ids_q=ids_q, ids_k=ids_k)
            return o[0]

        o_i = p_weighted(V64)
        absK = np.abs(K64)
        inner = abs(float(dO[i] @ o_i)) + float(np.abs(dO[i]) @ np.abs(o_i))
        terms = scale * (p_weighted(np.abs(V64 @ dO[i])[:, None] * absK) + inner * p_weighted(absK))
        err = np.abs(got[i] - want)
        worst = max(worst, float((err / (terms + 1e-30)).max()))
        assert (err <= TERMS_REL * terms + 1e-6).all(), (w.name, i, float((err / (terms + 1e-30)).max()))
    # ---- dV_j, dK_j of a few keys, element by element (one segment of the two smaller workloads) ------------
    if w.n <= 32768:
        keys = [3, w.n // 2 - 7, w.n // 2 + 250, w.n - 2] + [int(x) for x in inter["samples"][g, 0, :2].cpu().numpy()]   # two of them sampled columns of the root
        onehot = np.zeros((w.n, len(keys)))
        onehot[keys, np.arange(len(keys))] = 1.0
        Pcols, _ = O.segment_forward(Q64, K64, onehot, W, w.b, w.m, w.causal, w.n0, w.seed, g, scale=scale, ids_q=ids_q, ids_k=ids_k)
        O_all, _ = O.segment_forward(Q64, K64, V64, W, w.b, w.m, w.causal, w.n0, w.seed, g, scale=scale, ids_q=ids_q, ids_k=ids_k)
        delta = (dO * O_all).sum(axis=1)
        gv = dv.double().reshape(w.G, w.n, w.d)[g].cpu().numpy()
        gk = dk.double().reshape(w.G, w.n, w.d)[g].cpu().numpy()
        for c, j in enumerate(keys):
            P = Pcols[:, c]
            want_v = P @ dO
            size_v = P @ np.abs(dO)
            dS = P * (dO @ V64[j] - delta)
            want_k = scale * (dS @ Q64)
            size_k = scale * ((P * (np.abs(dO @ V64[j]) + np.abs(delta) + (np.abs(dO) * np.abs(O_all)).sum(axis=1))) @ np.abs(Q64))
            assert (np.abs(gv[j] - want_v) <= TERMS_REL * size_v + 1e-6).all(), (w.name, "dV", j)
            assert (np.abs(gk[j] - want_k) <= TERMS_REL * size_k + 1e-6).all(), (w.name, "dK", j)
    print(w.name, "dQ rows vs central differences: worst error / summed term sizes", worst,
          "sum dV error / size", sum_err / sum_size, "sum dK / size", dk_err / max(dk_size, 1e-30))
