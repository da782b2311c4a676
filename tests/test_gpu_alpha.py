"""The alpha of the paper's Theorem 1 (n times the largest squared column norm of the exact softmax matrix; Sec. 4.3
measures it on real models) computed on the GPU against the oracle, on synthetic inputs of the benchmark's kinds."""
import math

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

import parity_util as PU

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,d,kind,causal,skip,n_k", [(1000, 64, "gaussian", False, 0, 0), (2048, 128, "clustered", False, 0, 0),
                                                        (1537, 64, "gaussian", True, 32, 0), (1024, 128, "student_t", True, 0, 0),
                                                        (700, 64, "clustered", False, 5, 1900), (16, 64, "gaussian", True, 0, 0)])
def test_alpha_matches_the_oracle(n, d, kind, causal, skip, n_k):
    w = WL.Workload("alpha", 1, 3, n, d, "bf16", 64, 0, 4, causal, 64, kind, 90 + n, 0, n_k)
    arrs = WL.make_inputs(w)
    q, k, _ = PU.to_device(w, arrs)
    got = ha.alpha(q, k, causal=causal, skip_cols=skip).cpu().numpy().reshape(-1)
    Q64, K64 = WL.as_f64(arrs[0]), WL.as_f64(arrs[1])
    for g in range(w.G):
        ref = O.alpha_diagnostic(Q64[g], K64[g], 1.0 / math.sqrt(d), causal=causal, skip_cols=skip)
        # squared softmax weights from ex2.approx in fp32: a few 1e-6 relative per term, far inside 1e-3
        assert abs(got[g] - ref) <= 1e-3 * ref, (g, got[g], ref)
    print(kind, "n", n, "alpha", got, "alpha / n", got / n)
