"""The allocation-free sortLSH entry point.

Some users of the library cannot allocate device memory while they run (a server that splits
HBM between tenants at start-up, a plug-in inside another program's process, a control loop
that must never wait on the driver's allocator).  `hyperattn_sortlsh_noalloc` serves them with
scratch memory that lives inside the library image.  This test calls it through the C ABI twice in
a row and checks ids, permutation and inverse permutation bit for bit against what the ordinary
entry point (hyperattn_forward_ex with its exported intermediates) computes for the same rows,
and against the oracle's hash and stable argsort directly; it also checks that an oversized problem
is refused.  It is collected last on purpose."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2310_05869_b200 as ha
from paper_2310_05869_b200 import binding as B
from paper_2310_05869_b200 import workloads as WL
from oracle import hyperattn_oracle as O

pytestmark = pytest.mark.gpu


def _reference(x, hash_bits, seed):
    """ids / perm / rank of the rows of x from the ordinary forward call (x as queries and keys)."""
    n, d = x.shape
    q = x.view(1, 1, n, d)
    _, _, inter = ha.forward(q, q, q, block=min(128, n // 2), samples=0, hash_bits=hash_bits, seed=seed, debug=True)
    torch.cuda.synchronize()
    return inter["k_ids"][0], inter["perm_k"][0, 0], inter["rank_k"][0, 0]


@pytest.mark.parametrize("n,d,r,seed", [(4096, 64, 7, 0), (6144 + 256, 128, 8, 5), (4099, 64, 6, 2), (100, 128, 3, 1)])
def test_noalloc_matches_the_ordinary_entry_point_twice(n, d, r, seed):
    w = WL.Workload("noalloc", 1, 1, n, d, "bf16", 128, 0, r, False, 0, "clustered", 77, seed)
    bits = WL.make_inputs(w)[1][0]                                     # the key matrix: many equal ids
    x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    ref_ids, ref_perm, ref_rank = _reference(x, r, seed)
    # the oracle directly: ids up to hash bits whose projection is next to zero, the argsort of the GPU's ids exactly
    o_ids, absp = O.bucket_ids(WL.as_f64(bits), O.directions(d, r, seed))
    got_ids = ref_ids.cpu().numpy()
    for i in np.nonzero(o_ids != got_ids)[0]:
        diff = (int(o_ids[i]) ^ (int(o_ids[i]) >> 1)) ^ (int(got_ids[i]) ^ (int(got_ids[i]) >> 1))
        assert all(absp[i, t] < 1e-4 for t in range(r) if diff >> t & 1)
    o_perm, o_rank = O.stable_argsort(got_ids)
    for call in range(2):
        ids, perm, rank = ha.sortlsh_noalloc(x, r, seed)
        torch.cuda.synchronize()
        assert torch.equal(ids, ref_ids), f"ids differ on call {call}"
        assert torch.equal(perm, ref_perm), f"perm differs on call {call}"
        assert torch.equal(rank, ref_rank), f"rank differs on call {call}"
        assert (perm.cpu().numpy() == o_perm).all() and (rank.cpu().numpy() == o_rank).all()
    # a different matrix in between must not leave anything behind in the shared scratch
    y = torch.flip(x, dims=[0]).contiguous()
    ha.sortlsh_noalloc(y, r, seed)
    ids, perm, rank = ha.sortlsh_noalloc(x, r, seed)
    torch.cuda.synchronize()
    assert torch.equal(ids, ref_ids) and torch.equal(perm, ref_perm) and torch.equal(rank, ref_rank)


def test_noalloc_rejects_what_does_not_fit():
    x = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    out8 = torch.empty(128, dtype=torch.uint8, device="cuda")
    out32 = torch.empty(128, dtype=torch.int32, device="cuda")
    L = ha.lib()
    args = (out8.data_ptr(), out32.data_ptr(), out32.data_ptr(), None)
    assert L.hyperattn_sortlsh_noalloc(x.data_ptr(), B.NOALLOC_MAX_ROWS + 1, 64, 7, C.c_uint64(0), *args) == -2
    assert L.hyperattn_sortlsh_noalloc(x.data_ptr(), 128, 96, 7, C.c_uint64(0), *args) == -2
    assert L.hyperattn_sortlsh_noalloc(None, 128, 64, 7, C.c_uint64(0), *args) == -1
