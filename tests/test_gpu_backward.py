"""Backward pass against the oracle's dense form (derivative of the forward map with the sortLSH
permutations and the samples held fixed), on sizes whose n x n coefficient matrix fits in memory."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU

pytestmark = pytest.mark.gpu


def W(name, B, H, n, d, b, m, r, causal, n0, kind="gaussian", gen_seed=40, seed=0):
    return WL.Workload(name, B, H, n, d, "bf16", b, m, r, causal, n0, kind, gen_seed, seed)


CASES = [
    W("bwd_d64_blocks_and_samples", 1, 2, 1024, 64, 128, 64, 6, False, 0, seed=1),
    W("bwd_d128_blocks_and_samples", 1, 2, 1024, 128, 256, 128, 7, False, 0, seed=2),
    W("bwd_causal_two_levels_d64", 1, 2, 1024, 64, 64, 32, 5, True, 256, seed=3),
    W("bwd_causal_d128_ragged", 1, 1, 1536, 128, 96, 40, 6, True, 384, seed=4),
    W("bwd_exact_single_block", 1, 2, 300, 64, 512, 16, 4, False, 0, seed=5),
    W("bwd_causal_leaf_only", 1, 2, 500, 128, 64, 16, 4, True, 512, seed=6),
    W("bwd_clustered_duplicated_samples", 1, 1, 512, 64, 32, 200, 4, False, 0, kind="clustered", seed=7),
]

# Tolerance.  The weights P and dS enter the tensor cores as bf16 (relative rounding 2^-9 each, and dS is a
# product of two rounded factors), delta comes from the forward pass's bf16 output, and the sums run in fp32:
# an entry of a gradient can move by a few 2^-9 of the summed absolute values of its terms, which the oracle
# reports next to the gradients.  Bound: 2^-6 of that sum per entry (measured: up to 3 x 2^-9), and 2^-9 of
# its mean on average.  (A bound relative to the gradient itself would not hold where the terms cancel:
# clustered keys, sum_j dS_ij = 0.)
MAX_TERMS, MEAN_TERMS = 2.0 ** -6, 2.0 ** -9


def _random_cases(count):
    """Seeded draws of the forward pass's randomised shapes, kept to sizes whose dense form is quick."""
    import test_gpu_fuzz as F
    picked, s = [], 0
    while len(picked) < count:
        w = F.draw(1000 + s)
        s += 1
        if w.dtype == "bf16" and w.n <= 1600:
            picked.append(w.scaled(name=f"bwd_{w.name}_n{w.n}_d{w.d}_b{w.b}_m{w.m}_{'c' if w.causal else 'nc'}{w.n0}_{w.kind}", B=1, H=min(w.H, 2)))
    return picked


RANDOM = _random_cases(16)


@pytest.mark.parametrize("w", CASES + RANDOM, ids=[w.name for w in CASES + RANDOM])
def test_backward_matches_the_oracle(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, debug=True)
    rng = np.random.default_rng(900 + w.seed)
    dO = WL.f32_to_bf16_bits(rng.standard_normal((w.G, w.n, w.d)).astype(np.float32))
    dout = torch.from_numpy(dO.view(np.int16)).cuda().view(torch.bfloat16).view(w.B, w.H, w.n, w.d)
    dq, dk, dv = ha.backward(q, k, v, out, lse, dout, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed,
                             grad_dtype=torch.float32)
    dq16, dk16, dv16 = ha.backward(q, k, v, out, lse, dout, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (WL.as_f64(x) for x in arrs)
    dO64 = WL.as_f64(dO)
    gq = inter["q_ids"].cpu().numpy()
    gk = inter["k_ids"].cpu().numpy()
    scale = 1.0 / math.sqrt(w.d)
    for g in range(w.G):
        C = O.dense_coefficients(w.n, gq[g], gk[g], w.b, w.m, w.causal, w.n0, w.seed, g)
        ref, sizes = O.dense_backward(Q64[g], K64[g], V64[g], C, scale, dO64[g], with_term_sizes=True)
        for name, got, got16, want, size in zip("QKV", (dq, dk, dv), (dq16, dk16, dv16), ref, sizes):
            x = got.reshape(w.G, w.n, w.d)[g].double().cpu().numpy()
            top = np.abs(want).max()
            err = np.abs(x - want)
            assert np.isfinite(x).all()
            assert (err <= MAX_TERMS * size + 1e-6).all(), (name, g, float((err / (size + 1e-30)).max()))
            assert err.mean() <= MEAN_TERMS * size.mean(), (name, g, err.mean(), size.mean())
            x16 = got16.reshape(w.G, w.n, w.d)[g].float().cpu().numpy()
            assert np.abs(x16 - x).max() <= 2.0 ** -8 * max(top, np.abs(x).max()) + 1e-6    # the bf16 result is the rounded fp32 one (up to the order of the reductions)
            print(w.name, "d" + name, g, "max err / largest entry", err.max() / top, "max err / term sizes", float((err / (size + 1e-30)).max()))
