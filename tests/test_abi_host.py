"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, rejects bad arguments before touching the device, and its host-side helpers
agree with the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import binding as B
from oracle import hyperattn_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "hyperattn.h")).read()
    declared = set(re.findall(r"\b(hyperattn_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    L = ha.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert ha.version() >= 1


def test_status_strings():
    L = ha.lib()
    seen = {L.hyperattn_status_string(c).decode() for c in range(0, -7, -1)}
    assert len(seen) == 7 and "ok" in seen
    assert L.hyperattn_status_string(-99).decode() == "unknown status"


def _params(**kw):
    p = B._Params()
    base = dict(B=1, H=2, n=1024, d=64, block=128, samples=64, hash_bits=7, causal=0, n0=0, seed=0,
                dtype=B.BF16, out_dtype=B.BF16, softmax_scale=0.0)
    base.update(kw)
    for k, v in base.items():
        setattr(p, k, v)
    fake = 0x1000
    p.q, p.k, p.v, p.out, p.lse = fake, fake + 0x100000, fake + 0x200000, fake + 0x300000, fake + 0x400000
    return p


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), -2), (dict(hash_bits=0), -2), (dict(hash_bits=9), -2),
    (dict(block=0), -1), (dict(samples=-1), -1), (dict(B=0), -1), (dict(dtype=5), -1),
    (dict(causal=1, n0=0), -1), (dict(causal=1, n0=100, n=1000, n_k=900), -2), (dict(n_k=-5), -1),
    (dict(n=4096, block=1024, samples=256), -2),
])
def test_bad_shapes_are_rejected_on_the_host(kw, code):
    p = _params(**kw)
    assert ha.lib().hyperattn_forward_ex(C.byref(p)) == code
    nbytes = C.c_size_t(0)
    assert ha.lib().hyperattn_workspace_bytes(C.byref(p), C.byref(nbytes)) == code


def test_bad_pointers_are_rejected_on_the_host():
    L = ha.lib()
    p = _params(); p.q = None
    assert L.hyperattn_forward_ex(C.byref(p)) == -1
    p = _params(); p.k = 0x1008
    assert L.hyperattn_forward_ex(C.byref(p)) == -3
    p = _params(); p.out = p.v
    assert L.hyperattn_forward_ex(C.byref(p)) == -3
    assert L.hyperattn_forward_ex(None) == -1
    assert L.hyperattn_forward_host(None) == -1


def test_workspace_size_grows_with_the_problem():
    small = ha.workspace_bytes(1, 2, 1024, 64, 128, 64, 7)
    big = ha.workspace_bytes(1, 2, 4096, 64, 128, 64, 7)
    causal = ha.workspace_bytes(1, 2, 4096, 64, 128, 64, 7, True, 512)
    assert 0 < small < big < causal
    assert ha.workspace_bytes(1, 1, 256, 64, 256, 0, 7) <= 4096          # single block: nothing to sort


def test_projection_matrix_matches_the_oracle_bit_for_bit():
    for d, r, seed in [(64, 7, 0), (128, 8, 2 ** 40 + 17), (64, 1, 99)]:
        w = ha.get_projections(d, r, seed)
        ref = O.directions(d, r, seed)
        assert (w.view(np.uint32) == ref.view(np.uint32)).all()


def test_cuda_tensors_are_required():
    import torch
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16)
    with pytest.raises(ha.HyperAttnError):
        ha.forward(q, q, q, 64, 8, 4)


def test_binding_mirrors_the_stage_table_of_the_header():
    """The binding's stage-times structure must have the header's HYPERATTN_NUM_STAGES entries
    (hyperattn_profile_read writes that many)."""
    import re
    hdr = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "hyperattn.h")).read()
    n = int(re.search(r"HYPERATTN_NUM_STAGES\s*=\s*(\d+)", hdr).group(1))
    stages = re.findall(r"HYPERATTN_STAGE_(\w+)\s*=\s*(\d+)", hdr)
    from paper_2310_05869_b200 import binding as Bn
    assert Bn.NUM_STAGES == n == len(stages)
    assert [s.lower() for s, _ in sorted(stages, key=lambda t: int(t[1]))] == Bn.STAGE_NAMES


def test_backward_rejects_bad_arguments_on_the_host():
    """Nothing is launched for fp32 inputs, missing or misaligned gradient pointers, or a bad gradient type."""
    L = ha.lib()
    fake = 0x800000
    def grads(**kw):
        g = B._Grads(fake, fake + 0x100000, fake + 0x200000, fake + 0x300000, B.BF16)
        for k, v in kw.items():
            setattr(g, k, v)
        return g
    assert L.hyperattn_backward(C.byref(_params(dtype=B.FP32)), C.byref(grads())) == -2
    assert L.hyperattn_backward(C.byref(_params()), C.byref(grads(dq=0))) == -1
    assert L.hyperattn_backward(C.byref(_params()), C.byref(grads(grad_dtype=7))) == -1
    assert L.hyperattn_backward(C.byref(_params()), C.byref(grads(dk=fake + 0x100004))) == -3
    assert L.hyperattn_backward(None, C.byref(grads())) == -1
    need_f32, need_bf16, need_fwd = C.c_size_t(0), C.c_size_t(0), C.c_size_t(0)
    p = _params()
    assert L.hyperattn_backward_workspace_bytes(C.byref(p), B.FP32, C.byref(need_f32)) == 0
    assert L.hyperattn_backward_workspace_bytes(C.byref(p), B.BF16, C.byref(need_bf16)) == 0
    # bf16 gradients are accumulated in fp32 in the workspace: three tensors more than for fp32 gradients
    assert need_bf16.value - need_f32.value >= 3 * p.B * p.H * p.n * p.d * 4


def test_node_projections_match_the_oracle():
    for node in (0, 1, 7, 30):
        w = ha.get_projections(64, 7, 5, node=node)
        assert np.array_equal(w, O.directions(64, 7, 5, node=node))
    assert not np.array_equal(ha.get_projections(64, 7, 5, node=1), ha.get_projections(64, 7, 5))
