"""Randomised shapes: seeded draws over the whole argument space of the forward pass (sizes, block and
sample counts that divide nothing, hash widths, recursion depths, input kinds), each checked stage by
stage against the oracle like the hand-picked configurations."""
import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL

import parity_util as PU

pytestmark = pytest.mark.gpu


def draw(seed: int) -> WL.Workload:
    rng = np.random.default_rng(10_000 + seed)
    d = int(rng.choice([64, 128]))
    dtype = "fp32" if rng.random() < 0.1 else "bf16"
    B, H = int(rng.integers(1, 3)), int(rng.integers(1, 4))
    causal = bool(rng.random() < 0.5)
    n_k = 0
    ragged = 24 <= seed < 1000 and seed % 2 == 0      # (the draws above 1000 feed the backward tests: equal sides, lengths that 2^L divides)
    if causal:
        # 2^L leaves of any size: Alg. 4 halves until a part is not longer than n0
        leaf = int(np.exp(rng.uniform(np.log(3), np.log(1000))))
        L = int(rng.integers(0, 6))
        while leaf << L > 8192:
            L -= 1
        n = leaf << L
        n0 = int(rng.integers(leaf, 2 * leaf))
        if ragged:
            n = max(2, n - int(rng.integers(1, 1 << L)) if L else n)     # lengths that 2^L does not divide
    else:
        n0 = 0
        n = int(np.exp(rng.uniform(np.log(33), np.log(6000))))
        if ragged:
            n_k = int(np.exp(rng.uniform(np.log(33), np.log(6000))))     # queries and keys of different number
    while True:
        b = int(np.exp(rng.uniform(0, np.log(700))))
        m = int(rng.choice([0, int(np.exp(rng.uniform(0, np.log(600))))], p=[0.1, 0.9]))
        if 2 * ((b + 127) // 128 * 128) + (m + 127) // 128 * 128 <= 2048:
            break
    r = int(rng.integers(1, 9))
    kind = str(rng.choice(["gaussian", "clustered", "student_t", "ramp"], p=[0.4, 0.2, 0.2, 0.2]))
    return WL.Workload(f"fuzz{seed}", B, H, n, d, dtype, b, m, r, causal, n0, kind, 500 + seed, seed, n_k)


CASES = [draw(s) for s in range(40)]


def check(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    precise, bound = PU.output_policy(w, arrs)
    # every third draw asks for bf16 results (for bf16 inputs that also makes the partial rows of the causal recursion bf16)
    out_dtype = None if (w.seed % 3 == 0 and not precise) else torch.float32
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, out_dtype=out_dtype, debug=True,
                                 precise=precise)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (WL.as_f64(x) for x in arrs)
    if any(w.b < s for _, s in PU.levels_of(w)):
        amb, mism = PU.check_ids(w, Q64, K64, inter)
        assert mism <= amb
        PU.check_samples(w, inter)
        PU.check_perms(w, inter)
        return PU.check_outputs(w, Q64, K64, V64, out, lse, inter, max_abs_bound=bound)
    return PU.check_outputs(w, Q64, K64, V64, out, lse, None, max_abs_bound=bound)


@pytest.mark.parametrize("w", CASES, ids=[f"{w.name}_n{w.n}_k{w.nk}_d{w.d}_b{w.b}_m{w.m}_r{w.r}_{'c' if w.causal else 'nc'}{w.n0}_{w.kind}_{w.dtype}" for w in CASES])
def test_random_shapes(w):
    print(w, check(w))
