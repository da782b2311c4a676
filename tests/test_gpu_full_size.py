"""Parity at the full benchmark sizes, in the launch configuration the benchmark times.

The oracle cannot evaluate these workloads as a whole, so two segments (the first and the
last (batch, head) pair) are checked per workload: bucket ids and permutations in full, the
sampled columns of every segment, the outputs on the rows of 64 whole sorted blocks per checked
segment, on sampled rows and on the rows around every leaf boundary; every output of every
segment must be finite.  The 32768-row configuration is also compared row by row, all of it."""
import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import workloads as WL

import parity_util as PU

pytestmark = pytest.mark.gpu

# beyond the benchmark sizes: a million rows (eight recursion levels over 256 leaves) and half a million rows of d = 128
LONG = [WL.Workload("long_n1m_causal", 1, 2, 1048576, 64, "bf16", 256, 256, 7, True, 4096, "gaussian", 1010),
        WL.Workload("long_n512k_d128", 1, 1, 524288, 128, "bf16", 256, 256, 7, False, 0, "gaussian", 1011)]
# lengths that nothing divides, at size: a causal sequence of 100003 rows (32 leaves of 3126 rows, the last of 3097) and
# 50000 queries against 131072 keys
RAGGED = [WL.Workload("ragged_n100003_causal", 1, 4, 100003, 64, "bf16", 256, 256, 7, True, 4096, "gaussian", 1012),
          WL.Workload("ragged_cross_50000x131072", 1, 4, 50000, 64, "bf16", 256, 256, 7, False, 0, "gaussian", 1013, 0, 131072)]
FULL = [WL.CONFIGS[1], WL.CONFIGS[2], WL.CONFIGS[3], WL.CONFIGS[4]] + LONG + RAGGED


@pytest.mark.parametrize("w", FULL, ids=[w.name for w in FULL])
def test_full_size_sampled_segments(w):
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    precise, bound = PU.output_policy(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed, debug=True,
                                 out_dtype=torch.float32 if precise else None, precise=precise)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
    segs = [0, w.G - 1]
    Q64, K64, V64 = (PU.LazySegments(x) for x in arrs)
    amb, mism = PU.check_ids(w, Q64, K64, inter, segs=segs)
    assert mism <= amb
    PU.check_perms(w, inter, segs=segs)
    PU.check_samples(w, inter)
    stats = PU.check_outputs(w, Q64, K64, V64, out, lse, inter, rows_per_seg=48, segs=segs, rng_seed=1, max_abs_bound=bound,
                             blocks_per_seg=64)
    print(w.name, stats, "ambiguous hash bits", amb, "rows that differ", mism)


def test_c2_every_row_of_every_segment():
    """The 32768-row configuration (32 heads, d = 128) against the oracle on all of its 1 048 576 rows."""
    w = WL.CONFIGS[1]
    arrs = WL.make_inputs(w)
    q, k, v = PU.to_device(w, arrs)
    out, lse, inter = ha.forward(q, k, v, w.b, w.m, w.r, seed=w.seed, debug=True, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert ha.last_device_status() == 0
    Q64, K64, V64 = (PU.LazySegments(x) for x in arrs)
    amb, mism = PU.check_ids(w, Q64, K64, inter)
    assert mism <= amb
    PU.check_samples(w, inter)
    PU.check_perms(w, inter)
    stats = PU.check_outputs(w, Q64, K64, V64, out, lse, inter)
    assert stats["rows"] == w.G * w.n
    print(w.name, stats, "ambiguous hash bits", amb, "rows that differ", mism)
