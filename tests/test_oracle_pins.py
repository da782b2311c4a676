"""Pins for the CPU oracle: every stage is checked against something other than itself —
brute force on tiny inputs, closed forms, the paper's Fig. 1, published Philox vectors,
Monte-Carlo checks of Def. 1 and of the unbiased row-sum estimator of Alg. 2."""
import math
import os

import numpy as np
import pytest

from oracle import hyperattn_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ helpers (plain loops)
def brute_attention(Q, K, V, scale, causal):
    n, d = Q.shape
    out = np.zeros((n, V.shape[1]))
    lse = np.zeros(n)
    for i in range(n):
        tot = 0.0
        acc = [0.0] * V.shape[1]
        for j in range(K.shape[0]):
            if causal and j > i:
                continue
            s = 0.0
            for k in range(d):
                s += Q[i, k] * K[j, k]
            a = math.exp(scale * s)
            tot += a
            for c in range(V.shape[1]):
                acc[c] += a * V[j, c]
        out[i] = [x / tot for x in acc]
        lse[i] = math.log(tot)
    return out, lse


def rand_qkv(rng, n, d):
    return rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))


# ------------------------------------------------------------------ O8: random numbers
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for w in rows:
        v = [int(x, 16) for x in w]
        got = O.philox4x32_10(np.array(v[0:4]), (v[4], v[5]))
        assert [int(x) for x in got] == v[6:10]


def test_philox_vectorised_matches_scalar_calls():
    ctr = np.array([[i, 3, 5, 2] for i in range(17)])
    batch = O.philox4x32_10(ctr, (123, 456))
    for i in range(17):
        assert (O.philox4x32_10(ctr[i], (123, 456)) == batch[i]).all()


def test_directions_are_standard_normal():
    from scipy import stats
    W = O.directions(128, 8, 7).astype(np.float64).reshape(-1)
    W = np.concatenate([W, O.directions(128, 8, 8).astype(np.float64).reshape(-1)])
    assert abs(W.mean()) < 4 / math.sqrt(W.size)
    assert abs(W.var() - 1.0) < 4 * math.sqrt(2.0 / W.size)
    assert stats.kstest(W, "norm").pvalue > 1e-3
    # the (cos, sin) pairs of Box-Muller are uncorrelated and both halves are used
    assert abs(np.corrcoef(W[0::2], W[1::2])[0, 1]) < 0.1
    # prefix property: entry (k, t) is normal number k*r + t of one stream
    a = O.directions(4, 3, 5).reshape(-1)
    b = O.directions(8, 3, 5).reshape(-1)
    assert (a == b[:12]).all()
    assert O.directions(64, 7, 0).dtype == np.float32


def test_sample_indices_uniform_and_in_range():
    from scipy import stats
    N = 96
    s = np.concatenate([O.sample_indices(11, g, 3, 512, N) for g in range(40)])
    assert s.min() >= 0 and s.max() < N
    cnt = np.bincount(s, minlength=N)
    assert stats.chisquare(cnt).pvalue > 1e-3
    # streams of different segments / nodes / seeds differ; equal arguments repeat
    assert (O.sample_indices(1, 2, 3, 64, 1000) == O.sample_indices(1, 2, 3, 64, 1000)).all()
    assert (O.sample_indices(1, 2, 3, 64, 1000) != O.sample_indices(1, 2, 4, 64, 1000)).any()
    assert (O.sample_indices(1, 2, 3, 64, 1000) != O.sample_indices(1, 3, 3, 64, 1000)).any()
    assert (O.sample_indices(1, 2, 3, 64, 1000) != O.sample_indices(2, 2, 3, 64, 1000)).any()
    # floor(x N / 2^32) by hand for one word
    x = int(O.philox4x32_10(np.array([1, 2, 3, 2]), (1, 0))[2])
    assert int(O.sample_indices(1, 2, 3, 8, 1000)[6]) == (x * 1000) >> 32
    assert O.sample_indices(1, 2, 3, 0, 10).size == 0


# ------------------------------------------------------------------ O4: Def. 1
def test_gray_rank_adjacent_buckets_differ_in_one_sign():
    for r in range(1, 9):
        h = O.gray_rank(np.arange(1 << r), r)
        assert sorted(h.tolist()) == list(range(1 << r))          # a bijection
        inv = np.empty(1 << r, dtype=np.int64)
        inv[h] = np.arange(1 << r)                                # bucket id -> sign pattern
        for x in range(1 << r):
            assert x ^ (x >> 1) == inv[x]                         # the reflected Gray code
            diff = int(inv[x] ^ inv[(x + 1) % (1 << r)])
            assert bin(diff).count("1") == 1                      # cyclic adjacency


def test_bucket_bit_order_and_sign_convention():
    W = np.eye(3, dtype=np.float32)                               # direction t reads coordinate t
    X = np.array([[1.0, -1.0, -1.0],      # g = 001b = 1 -> h = 1
                  [1.0, 1.0, -1.0],       # g = 011b = 3 -> h = 2
                  [-1.0, 1.0, -1.0],      # g = 010b = 2 -> h = 3
                  [-1.0, -1.0, 1.0],      # g = 100b = 4 -> h = 7
                  [0.0, -0.0, 1.0]])      # zeros count as "not positive": g = 4 -> h = 7
    ids, absp = O.bucket_ids(X, W)
    assert ids.tolist() == [1, 2, 3, 7, 7]
    assert absp.shape == (5, 3) and absp[4, 0] == 0.0


def test_def1_collision_and_adjacency_probabilities():
    r, d, trials = 4, 6, 12000
    theta = 0.9
    x = np.zeros(d); x[0] = 2.0
    y = np.zeros(d); y[0] = 0.7 * math.cos(theta); y[1] = 0.7 * math.sin(theta)
    same = adj = 0
    for seed in range(trials):
        W = O.directions(d, r, seed)
        (hx, hy), _ = O.bucket_ids(np.stack([x, y]), W)
        hx, hy = int(hx), int(hy)
        same += hx == hy
        adj += (hy == (hx + 1) % (1 << r)) or (hy == (hx - 1) % (1 << r))
    p_same = (1 - theta / math.pi) ** r
    p_adj = (2 * theta / math.pi) * (1 - theta / math.pi) ** (r - 1)
    for got, p in ((same / trials, p_same), (adj / trials, p_adj)):
        assert abs(got - p) < 4 * math.sqrt(p * (1 - p) / trials), (got, p)


# ------------------------------------------------------------------ O7 / O5: sort and mask
def test_stable_argsort_against_python_sort():
    rng = np.random.default_rng(0)
    for n in (1, 2, 37, 500):
        ids = rng.integers(0, 9, size=n).astype(np.uint8)
        perm, rank = O.stable_argsort(ids)
        expect = [i for _, i in sorted((int(ids[i]), i) for i in range(n))]
        assert perm.tolist() == expect
        assert all(rank[perm[p]] == p for p in range(n))


def test_fig1_mask():
    spec = {}
    for line in open(os.path.join(GOLDEN, "fig1_sortlsh.txt")):
        if line.strip() and line[0] != "#":
            k, *v = line.split()
            spec[k] = v
    sq = [int(x) - 1 for x in spec["sorted_queries"]]
    sk = [int(x) - 1 for x in spec["sorted_keys"]]
    b = int(spec["block"][0])
    boxed = {tuple(int(t) - 1 for t in e.split("-")) for e in spec["boxed"]}
    assert len(boxed) == 23
    # bucket ids that reproduce the printed order (one row per bucket)
    ids_q = np.empty(9, dtype=np.uint8); ids_q[sq] = np.arange(9)
    ids_k = np.empty(9, dtype=np.uint8); ids_k[sk] = np.arange(9)
    perm_q, rank_q = O.stable_argsort(ids_q)
    perm_k, rank_k = O.stable_argsort(ids_k)
    assert perm_q.tolist() == sq and perm_k.tolist() == sk
    M = O.sortlsh_mask(rank_q, rank_k, b)
    assert M.sum() == 27 and (M.sum(axis=0) == 3).all() and (M.sum(axis=1) == 3).all()
    assert all(M[i, j] == 1 for i, j in boxed)
    # the three diagonal blocks of the middle panel
    for blk in range(3):
        for i in sq[3 * blk:3 * blk + 3]:
            assert sorted(np.nonzero(M[i])[0].tolist()) == sorted(sk[3 * blk:3 * blk + 3])


# ------------------------------------------------------------------ O1: exact attention
@pytest.mark.parametrize("causal", [False, True])
def test_exact_attention_brute_force(causal):
    rng = np.random.default_rng(1)
    Q, K, V = rand_qkv(rng, 13, 5)
    out, lse = O.exact_attention(Q, K, V, 0.37, causal=causal)
    bo, bl = brute_attention(Q, K, V, 0.37, causal)
    np.testing.assert_allclose(out, bo, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, bl, rtol=0, atol=1e-12)
    o2, l2 = O.exact_attention(Q, K, V, 0.37, causal=causal, rows=[12, 0, 5])
    np.testing.assert_allclose(o2, bo[[12, 0, 5]], atol=1e-12)
    np.testing.assert_allclose(l2, bl[[12, 0, 5]], atol=1e-12)


def test_single_block_is_exact_attention():
    """b = N (or b > N): the mask is all ones, nothing is sampled."""
    rng = np.random.default_rng(2)
    Q, K, V = (x[None] for x in rand_qkv(rng, 24, 4))
    bo, bl = brute_attention(Q[0], K[0], V[0], 0.5, False)
    for b in (24, 64):
        out, lse = O.forward(Q, K, V, b=b, m=8, r=3, seed=4, scale=0.5)
        np.testing.assert_allclose(out[0], bo, atol=1e-12)
        np.testing.assert_allclose(lse[0], bl, atol=1e-12)


def test_causal_base_case_is_exact_causal_attention():
    rng = np.random.default_rng(3)
    Q, K, V = (x[None] for x in rand_qkv(rng, 16, 4))
    bo, bl = brute_attention(Q[0], K[0], V[0], 0.5, True)
    out, lse = O.forward(Q, K, V, b=4, m=4, r=3, causal=True, n0=16, seed=4, scale=0.5)
    np.testing.assert_allclose(out[0], bo, atol=1e-12)
    np.testing.assert_allclose(lse[0], bl, atol=1e-12)


# ------------------------------------------------------------------ O2: causal bookkeeping
@pytest.mark.parametrize("n,n0", [(32, 4), (32, 8), (48, 12), (64, 2), (48, 5), (40, 7), (72, 10)])   # the last three: leaves of 3, 5 and 9 rows (n0 does not divide n)
def test_causal_recursion_with_single_block_nodes_is_exact(n, n0):
    """With b >= n/2 every off-diagonal problem is one block, so Alg. 4's identity
    D_C = diag(D_C11, D_21 + D_C22) must give exact causal attention for any depth."""
    rng = np.random.default_rng(n + n0)
    Q, K, V = (x[None] for x in rand_qkv(rng, n, 3))
    bo, bl = brute_attention(Q[0], K[0], V[0], 0.6, True)
    out, lse = O.forward(Q, K, V, b=n // 2, m=8, r=4, causal=True, n0=n0, seed=1, scale=0.6)
    np.testing.assert_allclose(out[0], bo, atol=1e-11)
    np.testing.assert_allclose(lse[0], bl, atol=1e-11)


# ------------------------------------------------------------------ residual path: closed forms
def test_samples_covering_every_key_once_give_exact_attention():
    """m = N samples hitting each key exactly once: N/m = 1, the off-block sum is complete,
    so masked + residual is the full row sum and the output is exact attention."""
    rng = np.random.default_rng(5)
    N, b = 32, 8
    Q, K, V = rand_qkv(rng, N, 6)
    iq = rng.integers(0, 8, N).astype(np.uint8)
    ik = rng.integers(0, 8, N).astype(np.uint8)
    out, lse = O.node_forward(Q, K, V, iq, ik, rng.permutation(N), b, 0.4)
    bo, bl = brute_attention(Q, K, V, 0.4, False)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)


def test_zero_logits_give_counting_closed_form():
    """Q = 0 makes every attention entry 1: d~_i = b + (N/m) #{t : l_t outside i's block};
    V = 1 makes every output exactly 1 (weights sum to one)."""
    rng = np.random.default_rng(6)
    N, b, m, d = 40, 8, 12, 3
    K = rng.standard_normal((N, d))
    iq = rng.integers(0, 16, N).astype(np.uint8)
    ik = rng.integers(0, 16, N).astype(np.uint8)
    smp = rng.integers(0, N, m)
    out, lse = O.node_forward(np.zeros((N, d)), K, np.ones((N, d)), iq, ik, smp, b, 1.0)
    order_q = sorted(range(N), key=lambda i: (int(iq[i]), i))
    order_k = sorted(range(N), key=lambda i: (int(ik[i]), i))
    for i in range(N):
        beta = order_q.index(i) // b
        outside = sum(1 for l in smp if order_k.index(int(l)) // b != beta)
        assert abs(lse[i] - math.log(b + (N / m) * outside)) < 1e-12
    np.testing.assert_allclose(out, 1.0, atol=1e-12)


def test_ragged_last_block_counting_closed_form_and_full_coverage():
    """N not a multiple of b: the mask of Alg. 1 line 4 is floor(P(i)/b), so the last sorted block
    has N mod b rows.  Q = 0 gives d~_i = |block of i| + (N/m) #{t : l_t outside i's block};
    samples covering every key once give exact attention, whatever the block sizes."""
    rng = np.random.default_rng(16)
    N, b, m, d = 37, 8, 11, 3                                   # blocks of 8, 8, 8, 8, 5
    K = rng.standard_normal((N, d))
    iq = rng.integers(0, 16, N).astype(np.uint8)
    ik = rng.integers(0, 16, N).astype(np.uint8)
    smp = rng.integers(0, N, m)
    out, lse = O.node_forward(np.zeros((N, d)), K, np.ones((N, d)), iq, ik, smp, b, 1.0)
    order_q = sorted(range(N), key=lambda i: (int(iq[i]), i))
    order_k = sorted(range(N), key=lambda i: (int(ik[i]), i))
    for i in range(N):
        beta = order_q.index(i) // b
        size = sum(1 for j in range(N) if order_k.index(j) // b == beta)
        assert size == (5 if beta == 4 else 8)
        outside = sum(1 for l in smp if order_k.index(int(l)) // b != beta)
        assert abs(lse[i] - math.log(size + (N / m) * outside)) < 1e-12
    np.testing.assert_allclose(out, 1.0, atol=1e-12)
    Q, K, V = rand_qkv(rng, N, 5)
    out, lse = O.node_forward(Q, K, V, iq, ik, rng.permutation(N), b, 0.4)
    bo, bl = brute_attention(Q, K, V, 0.4, False)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)


@pytest.mark.parametrize("causal,n,n0,b", [(False, 26, 0, 4), (True, 24, 6, 5)])
def test_dense_weights_with_ragged_blocks(causal, n, n0, b):
    """The dense cross-form stays row-stochastic and reproduces the output when block sizes do
    not divide the node sizes (causal: nodes of 12 and 6 rows with b = 5)."""
    rng = np.random.default_rng(17)
    d, m, r, seed, scale = 4, 5, 3, 33, 0.5
    Q, K, V = rand_qkv(rng, n, d)
    W = O.directions(d, r, seed)
    iq, _ = O.bucket_ids(Q, W)
    ik, _ = O.bucket_ids(K, W)
    Wt = O.dense_weights(Q, K, iq, ik, b, m, scale, causal, n0, seed, g=1)
    np.testing.assert_allclose(Wt.sum(axis=1), 1.0, atol=1e-12)
    if causal:
        assert np.triu(Wt, 1).max() == 0.0
    out, _ = O.segment_forward(Q, K, V, W, b, m, causal, n0, seed, g=1, scale=scale)
    np.testing.assert_allclose(out, Wt @ V, atol=1e-12)


def test_no_samples_and_all_colliding_samples():
    rng = np.random.default_rng(7)
    N, b = 16, 4
    Q, K, V = rand_qkv(rng, N, 3)
    ids = np.repeat(np.arange(4), 4).astype(np.uint8)            # blocks = consecutive rows
    out0, lse0 = O.node_forward(Q, K, V, ids, ids, np.zeros(0, dtype=int), b, 0.5)
    for blk in range(4):
        sl = slice(4 * blk, 4 * blk + 4)
        bo, bl = brute_attention(Q[sl], K[sl], V[sl], 0.5, False)
        np.testing.assert_allclose(out0[sl], bo, atol=1e-12)
        np.testing.assert_allclose(lse0[sl], bl, atol=1e-12)
    # samples all inside block 0: rows of block 0 see no residual at all
    out1, lse1 = O.node_forward(Q, K, V, ids, ids, np.array([0, 1, 2, 3]), b, 0.5)
    np.testing.assert_allclose(out1[:4], out0[:4], atol=1e-12)
    np.testing.assert_allclose(lse1[:4], lse0[:4], atol=1e-12)
    assert (lse1[4:] > lse0[4:]).all()


# ------------------------------------------------------------------ O6: unbiased estimator
def test_sampled_row_sum_and_numerator_are_unbiased():
    """Alg. 2 line 7 (uncapped): E[(N/m) sum_t (1 - M_{i,l_t}) A_{i,l_t}] is the off-block row
    sum; with the same weights on V the numerator's expectation is (A V)_i."""
    rng = np.random.default_rng(8)
    N, b, m, d, scale = 24, 6, 5, 3, 0.3
    Q, K, V = rand_qkv(rng, N, d)
    iq = rng.integers(0, 8, N).astype(np.uint8)
    ik = rng.integers(0, 8, N).astype(np.uint8)
    trials = 6000
    dens = np.zeros((trials, N))
    nums = np.zeros((trials, N, d))
    for t in range(trials):
        smp = O.sample_indices(t, 0, 0, m, N)
        out, lse = O.node_forward(Q, K, V, iq, ik, smp, b, scale)
        dens[t] = np.exp(lse)
        nums[t] = out * dens[t][:, None]
    A = np.exp(scale * Q @ K.T)
    full_den = A.sum(axis=1)
    full_num = A @ V
    se_d = dens.std(axis=0, ddof=1) / math.sqrt(trials)
    se_n = nums.std(axis=0, ddof=1) / math.sqrt(trials)
    assert (np.abs(dens.mean(axis=0) - full_den) < 4.5 * se_d).all()
    assert (np.abs(nums.mean(axis=0) - full_num) < 4.5 * se_n + 1e-12).all()
    assert (se_d > 0).all()                                       # the sampled term is really there


# ------------------------------------------------------------------ O3: dense cross-form
@pytest.mark.parametrize("causal,n0", [(False, 0), (True, 8), (True, 4)])
def test_dense_weights_are_row_stochastic_and_reproduce_output(causal, n0):
    rng = np.random.default_rng(9)
    n, d, b, m, r, seed, scale = 32, 4, 4, 6, 3, 21, 0.45
    Q, K, V = rand_qkv(rng, n, d)
    W = O.directions(d, r, seed)
    iq, _ = O.bucket_ids(Q, W)
    ik, _ = O.bucket_ids(K, W)
    Wt = O.dense_weights(Q, K, iq, ik, b, m, scale, causal, n0, seed, g=2)
    np.testing.assert_allclose(Wt.sum(axis=1), 1.0, atol=1e-12)
    assert (Wt >= 0).all()
    if causal:
        assert np.triu(Wt, 1).max() == 0.0
    out, lse = O.segment_forward(Q, K, V, W, b, m, causal, n0, seed, g=2, scale=scale)
    np.testing.assert_allclose(out, Wt @ V, atol=1e-12)
    # V = ones gives ones
    out1, _ = O.segment_forward(Q, K, np.ones_like(V), W, b, m, causal, n0, seed, g=2, scale=scale)
    np.testing.assert_allclose(out1, 1.0, atol=1e-12)
    # rows can be evaluated in any subset / order
    rows = np.array([31, 0, 17, 8, 16])
    o2, l2 = O.segment_forward(Q, K, V, W, b, m, causal, n0, seed, g=2, scale=scale, rows=rows)
    np.testing.assert_allclose(o2, out[rows], atol=1e-13)
    np.testing.assert_allclose(l2, lse[rows], atol=1e-13)


def test_causal_nodes_use_their_own_sample_streams():
    """Second-quarter rows of a two-level recursion only see node 1 (left child) and
    the leaves; last-quarter rows see node 0 and node 2."""
    rng = np.random.default_rng(10)
    n, d, b, m, r, seed, scale, n0 = 32, 4, 2, 4, 3, 3, 0.5, 8
    Q, K, V = rand_qkv(rng, n, d)
    W = O.directions(d, r, seed)
    iq, _ = O.bucket_ids(Q, W)
    ik, _ = O.bucket_ids(K, W)
    out, lse = O.segment_forward(Q, K, V, W, b, m, True, n0, seed, g=0, scale=scale)
    # rebuild rows 8..15 by hand: exact causal on [8,16) merged with node 1 on (Q[8:16], K[:8])
    o22, l22 = O.exact_attention(Q[8:16], K[8:16], V[8:16], scale, causal=True)
    smp = O.sample_indices(seed, 0, O.heap_node(1, 0), m, 8)
    o21, l21 = O.node_forward(Q[8:16], K[:8], V[:8], iq[8:16], ik[:8], smp, b, scale)
    den = np.exp(l21) + np.exp(l22)
    np.testing.assert_allclose(lse[8:16], np.log(den), atol=1e-12)
    np.testing.assert_allclose(out[8:16], (o21 * np.exp(l21)[:, None] + o22 * np.exp(l22)[:, None]) / den[:, None],
                               atol=1e-12)


# ------------------------------------------------------------------ O9: permutation invariance
def test_joint_permutation_of_keys_and_values_single_block():
    rng = np.random.default_rng(11)
    Q, K, V = rand_qkv(rng, 20, 4)
    p = rng.permutation(20)
    ids = rng.integers(0, 4, 20).astype(np.uint8)
    a, la = O.node_forward(Q, K, V, ids, ids, [], 20, 0.5)
    c, lc = O.node_forward(Q, K[p], V[p], ids, ids[p], [], 20, 0.5)
    np.testing.assert_allclose(a, c, atol=1e-12)
    np.testing.assert_allclose(la, lc, atol=1e-12)


# ---- backward pass: the derivative of the forward map, discrete choices held fixed --------------
@pytest.mark.parametrize("causal,n,n0,b,m", [(False, 48, 0, 8, 6), (True, 64, 16, 8, 5), (False, 40, 0, 64, 0), (True, 32, 32, 4, 4)])
def test_backward_matches_finite_differences_of_the_forward_oracle(causal, n, n0, b, m):
    """Central differences of the (independently written) forward oracle along random directions,
    with the bucket ids injected so that the sortLSH permutations do not move."""
    rng = np.random.default_rng(77 + n + b)
    d, r, seed, g = 8, 4, 3, 1
    Q, K, V = (rng.standard_normal((n, d)) for _ in range(3))
    W = O.directions(d, r, seed)
    ids_q, _ = O.bucket_ids(Q, W)
    ids_k, _ = O.bucket_ids(K, W)
    scale = 0.4
    G_out = rng.standard_normal((n, d))
    g_lse = rng.standard_normal(n)

    def loss(Q_, K_, V_):
        out, lse = O.segment_forward(Q_, K_, V_, W, b, m, causal, n0, seed, g, scale=scale, ids_q=ids_q, ids_k=ids_k)
        return float((out * G_out).sum() + (lse * g_lse).sum())

    C = O.dense_coefficients(n, ids_q, ids_k, b, m, causal, n0, seed, g)
    dQ, dK, dV = O.dense_backward(Q, K, V, C, scale, G_out, g_lse)
    eps = 1e-6
    for X, dX, which in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2)):
        for _ in range(3):
            D = rng.standard_normal(X.shape)
            args_p = [Q, K, V]; args_m = [Q, K, V]
            args_p[which] = X + eps * D; args_m[which] = X - eps * D
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            an = float((dX * D).sum())
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (which, fd, an)


def test_dense_coefficients_reproduce_dense_weights():
    rng = np.random.default_rng(5)
    n, d, r, b, m, seed, g = 64, 8, 5, 8, 7, 11, 2
    Q, K = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    W = O.directions(d, r, seed)
    ids_q, _ = O.bucket_ids(Q, W)
    ids_k, _ = O.bucket_ids(K, W)
    for causal, n0 in ((False, 0), (True, 16)):
        C = O.dense_coefficients(n, ids_q, ids_k, b, m, causal, n0, seed, g)
        U = C * np.exp(0.3 * (Q @ K.T))
        Wt = O.dense_weights(Q, K, ids_q, ids_k, b, m, 0.3, causal, n0, seed, g)
        assert np.allclose(U / U.sum(axis=1, keepdims=True), Wt, rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ unequal sides, lengths the split does not divide
def brute_node(Q, K, V, iq, ik, smp, b, b_q, scale):
    """Alg. 2 lines 7 and 9 (no caps) with explicit loops: query i belongs to group floor(P_Q(i)/b_q), key j
    to group floor(P_K(j)/b); the positions come from Python's stable sort."""
    n_q, N = Q.shape[0], K.shape[0]
    order_q = sorted(range(n_q), key=lambda i: (int(iq[i]), i))
    order_k = sorted(range(N), key=lambda j: (int(ik[j]), j))
    pos_q = {i: p for p, i in enumerate(order_q)}
    pos_k = {j: p for p, j in enumerate(order_k)}
    m = len(smp)
    out = np.zeros((n_q, V.shape[1]))
    lse = np.zeros(n_q)
    for i in range(n_q):
        beta = pos_q[i] // b_q
        den, num = 0.0, np.zeros(V.shape[1])
        for j in range(N):
            if pos_k[j] // b == beta:
                a = math.exp(scale * float(Q[i] @ K[j]))
                den += a
                num += a * V[j]
        for l in smp:
            if pos_k[int(l)] // b != beta:
                a = (N / m) * math.exp(scale * float(Q[i] @ K[int(l)]))
                den += a
                num += a * V[int(l)]
        out[i] = num / den
        lse[i] = math.log(den)
    return out, lse


def test_query_block_size_rule():
    """b_q = ceil(b n_q / n_k): equal sides keep b; the hand-worked case n_q = 5, n_k = 10, b = 4 gives groups
    of 2 queries against groups of 4 keys; there is never a query group without a key group."""
    assert O.query_block_size(10, 10, 4) == 4 and O.query_block_size(37, 37, 8) == 8
    assert O.query_block_size(5, 10, 4) == 2 and O.query_block_size(20, 10, 4) == 8
    assert O.query_block_size(4095, 4096, 256) == 256            # the causal case: sides that differ by a few rows
    rng = np.random.default_rng(0)
    for _ in range(2000):
        n_q, n_k, b = int(rng.integers(1, 500)), int(rng.integers(2, 500)), int(rng.integers(1, 300))
        if b >= n_k:
            continue
        b_q = O.query_block_size(n_q, n_k, b)
        assert b_q >= 1 and -(-n_q // b_q) <= -(-n_k // b)
    # the hand-worked mask: sorted queries 0..4 -> groups 0 0 1 1 2, sorted keys 0..9 -> groups 0 0 0 0 1 1 1 1 2 2
    M = O.sortlsh_mask(np.arange(5), np.arange(10), 4, 2)
    want = np.zeros((5, 10), dtype=int)
    want[0:2, 0:4] = 1; want[2:4, 4:8] = 1; want[4, 8:10] = 1
    assert (M == want).all()


@pytest.mark.parametrize("n_q,n_k,b,m", [(13, 40, 8, 9), (50, 21, 6, 7), (5, 10, 4, 3), (31, 32, 8, 5)])
def test_unequal_sides_against_explicit_loops(n_q, n_k, b, m):
    rng = np.random.default_rng(n_q * 100 + n_k)
    Q = rng.standard_normal((n_q, 4)); K = rng.standard_normal((n_k, 4)); V = rng.standard_normal((n_k, 3))
    iq = rng.integers(0, 6, n_q).astype(np.uint8); ik = rng.integers(0, 6, n_k).astype(np.uint8)
    smp = rng.integers(0, n_k, m)
    out, lse = O.node_forward(Q, K, V, iq, ik, smp, b, 0.5)
    bo, bl = brute_node(Q, K, V, iq, ik, smp, b, -(-b * n_q // n_k), 0.5)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)
    # a subset of rows gives the same rows
    rows = np.array(sorted(rng.choice(n_q, size=min(4, n_q), replace=False)))
    o2, l2 = O.node_forward(Q, K, V, iq, ik, smp, b, 0.5, rows=rows)
    np.testing.assert_allclose(o2, out[rows], atol=1e-14)
    np.testing.assert_allclose(l2, lse[rows], atol=1e-14)


@pytest.mark.parametrize("n_q,n_k,b", [(13, 40, 8), (50, 21, 6)])
def test_unequal_sides_full_coverage_is_exact_and_dense_form_is_row_stochastic(n_q, n_k, b):
    rng = np.random.default_rng(n_q + n_k)
    Q = rng.standard_normal((n_q, 5)); K = rng.standard_normal((n_k, 5)); V = rng.standard_normal((n_k, 4))
    W = O.directions(5, 3, 9)
    iq, _ = O.bucket_ids(Q, W); ik, _ = O.bucket_ids(K, W)
    out, lse = O.node_forward(Q, K, V, iq, ik, rng.permutation(n_k), b, 0.4)      # every key sampled once
    bo, bl = brute_attention(Q, K, V, 0.4, False)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)
    # the whole forward with its own samples: the implied weights are row-stochastic and give the output
    o, l = O.segment_forward(Q, K, V, W, b, 7, False, 0, 3, 2, scale=0.4)
    Wd = O.dense_weights(Q, K, iq, ik, b, 7, 0.4, False, 0, 3, 2)
    assert Wd.shape == (n_q, n_k)
    np.testing.assert_allclose(Wd.sum(axis=1), 1.0, atol=1e-12)
    np.testing.assert_allclose(Wd @ V, o, atol=1e-12)


def test_causal_grid():
    assert O.causal_grid(131072, 4096) == (5, 4096) and O.causal_grid(4096, 4096) == (0, 4096)
    assert O.causal_grid(6000, 1000) == (3, 750) and O.causal_grid(100003, 4096) == (5, 3126)
    assert O.causal_grid(5, 2) == (2, 2) and O.causal_grid(7, 1) == (3, 1)


@pytest.mark.parametrize("n,n0", [(33, 4), (47, 6), (101, 9), (5, 2), (7, 1), (100, 7), (19, 32)])
def test_causal_lengths_the_split_does_not_divide_single_block_nodes_are_exact(n, n0):
    """Any n: with b at least the largest off-diagonal problem every node is one block, and the recursion
    over a short last leaf and short last nodes must still add up to exact causal attention."""
    rng = np.random.default_rng(n * 7 + n0)
    Q, K, V = (x[None] for x in rand_qkv(rng, n, 3))
    bo, bl = brute_attention(Q[0], K[0], V[0], 0.6, True)
    out, lse = O.forward(Q, K, V, b=n, m=8, r=4, causal=True, n0=n0, seed=1, scale=0.6)
    np.testing.assert_allclose(out[0], bo, atol=1e-11)
    np.testing.assert_allclose(lse[0], bl, atol=1e-11)


@pytest.mark.parametrize("n,n0,b,m", [(45, 6, 4, 5), (101, 13, 5, 6), (37, 5, 3, 4)])
def test_causal_odd_lengths_dense_form_and_rebuilt_last_node(n, n0, b, m):
    """Sorted nodes with a short last node: the implied weights are row-stochastic, lower triangular and give the
    output; the rows of the last (short) root-level node are rebuilt by hand from node_forward and the
    recursion on the second part."""
    rng = np.random.default_rng(n)
    Q, K, V = rand_qkv(rng, n, 4)
    W = O.directions(4, 3, 5)
    iq, _ = O.bucket_ids(Q, W); ik, _ = O.bucket_ids(K, W)
    out, lse = O.segment_forward(Q, K, V, W, b, m, True, n0, 11, 1, scale=0.7)
    Wd = O.dense_weights(Q, K, iq, ik, b, m, 0.7, True, n0, 11, 1)
    np.testing.assert_allclose(Wd.sum(axis=1), 1.0, atol=1e-12)
    assert np.abs(np.triu(Wd, 1)).max() == 0.0
    np.testing.assert_allclose(Wd @ V, out, atol=1e-12)
    L, leaf = O.causal_grid(n, n0)
    h = (leaf << L) // 2                                          # the root splits at half of the rounded-up length
    assert h < n < 2 * h or n == 2 * h
    smp = O.sample_indices(11, 1, 0, m if b < h else 0, h)
    o21, l21 = O.node_forward(Q[h:], K[:h], V[:h], iq[h:], ik[:h], smp, b, 0.7)
    # total row sum of a second-part row = its off-diagonal estimate + everything the recursion gives it inside the second part
    inside = np.log(np.exp(lse[h:]) - np.exp(l21))
    C = O.dense_coefficients(n, iq, ik, b, m, True, n0, 11, 1)
    A = np.exp(0.7 * (Q @ K.T))
    np.testing.assert_allclose(np.log((C * A)[h:, h:].sum(axis=1)), inside, atol=1e-9)
    np.testing.assert_allclose(np.log((C * A)[h:, :h].sum(axis=1)), l21, atol=1e-12)


# ------------------------------------------------------------------ Alg. 2 with its caps
def brute_capped(Q, K, V, iq, ik, smp, T, b, scale, cap_scale, kappa):
    """Alg. 2 lines 3, 6, 7, 9 with explicit loops, in plain exp arithmetic (small logits)."""
    n_q, N = Q.shape[0], K.shape[0]
    b_q = -(-b * n_q // N)
    order_q = sorted(range(n_q), key=lambda i: (int(iq[i]), i))
    order_k = sorted(range(N), key=lambda j: (int(ik[j]), j))
    pos_q = {i: p for p, i in enumerate(order_q)}
    pos_k = {j: p for p, j in enumerate(order_k)}
    m = len(smp)
    A = [[math.exp(scale * float(Q[i] @ K[j])) for j in range(N)] for i in range(n_q)]
    inside = lambda i, j: pos_k[j] // b == pos_q[i] // b_q
    tau = max([sum(A[order_q[p]][k] for k in range(N) if not inside(order_q[p], k)) for p in T], default=0.0)       # line 3 (T: sorted positions)
    out = np.zeros((n_q, V.shape[1]))
    lse = np.zeros(n_q)
    for i in range(n_q):
        masked = sum(A[i][j] for j in range(N) if inside(i, j))
        C = cap_scale * m / (N * math.log(N)) * (masked + tau / kappa)                                # line 6
        d = (N / m) * sum(min(A[i][int(l)], C) for l in smp if not inside(i, int(l)))                 # line 7
        dt = masked + max(d, tau / kappa)                                                             # line 9
        num = sum(A[i][j] * V[j] for j in range(N) if inside(i, j))
        num = num + (N / m) * sum((A[i][int(l)] * V[int(l)] for l in smp if not inside(i, int(l))), np.zeros(V.shape[1]))
        out[i] = num / dt
        lse[i] = math.log(dt)
    return out, lse, tau


@pytest.mark.parametrize("cap_scale,kappa", [(3.0, 2.0), (40.0, 50.0), (0.5, 1000.0)])
def test_capped_row_sums_against_explicit_loops(cap_scale, kappa):
    rng = np.random.default_rng(int(cap_scale * 10 + kappa))
    N, b, m, d = 36, 6, 9, 4
    Q, K, V = rand_qkv(rng, N, d)
    iq = rng.integers(0, 8, N).astype(np.uint8); ik = rng.integers(0, 8, N).astype(np.uint8)
    smp = rng.integers(0, N, m); T = rng.integers(0, N, m)
    out, lse = O.node_forward(Q, K, V, iq, ik, smp, b, 0.8, caps=(cap_scale, kappa, T))
    bo, bl, tau = brute_capped(Q, K, V, iq, ik, smp, T, b, 0.8, cap_scale, kappa)
    np.testing.assert_allclose(lse, bl, atol=1e-11)
    np.testing.assert_allclose(out, bo, atol=1e-11)
    # and the caps did something in at least one of the parameter sets: the result differs from the uncapped one
    o0, l0 = O.node_forward(Q, K, V, iq, ik, smp, b, 0.8)
    if cap_scale < 10:
        assert np.abs(l0 - lse).max() > 1e-6


def test_caps_switched_off_reproduce_the_uncapped_path_bit_for_bit():
    rng = np.random.default_rng(77)
    Q, K, V = (x[None] for x in rand_qkv(rng, 96, 5))
    for causal, n0 in ((False, 0), (True, 12)):
        o0, l0 = O.forward(Q, K, V, b=8, m=10, r=4, causal=causal, n0=n0, seed=3, scale=0.5)
        o1, l1 = O.forward(Q, K, V, b=8, m=10, r=4, causal=causal, n0=n0, seed=3, scale=0.5, caps=(math.inf, math.inf))
        assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


def test_capped_zero_logits_closed_form_with_a_binding_cap_and_the_lower_cap():
    """Q = 0: every entry is 1, the masked sum of a row is its block's size, tau = N - (smallest block size among
    the rows of T), and a cap below 1 binds on every sampled entry."""
    rng = np.random.default_rng(8)
    N, b, m, d = 37, 8, 12, 3                                      # blocks of 8, 8, 8, 8, 5
    K = rng.standard_normal((N, d)); V = np.ones((N, d))
    iq = rng.integers(0, 16, N).astype(np.uint8); ik = rng.integers(0, 16, N).astype(np.uint8)
    smp = rng.integers(0, N, m); T = np.arange(N)                   # every row: tau = N - 5 (a row of the short block)
    cap_scale, kappa = 0.3, 4.0
    out, lse = O.node_forward(np.zeros((N, d)), K, V, iq, ik, smp, b, 1.0, caps=(cap_scale, kappa, T))
    order_q = sorted(range(N), key=lambda i: (int(iq[i]), i))
    order_k = sorted(range(N), key=lambda i: (int(ik[i]), i))
    tau = N - 5
    for i in range(N):
        beta = order_q.index(i) // b
        blk = min(b, N - beta * b)
        outside = sum(1 for l in smp if order_k.index(int(l)) // b != beta)
        C = cap_scale * m / (N * math.log(N)) * (blk + tau / kappa)
        assert C < 1.0                                              # the cap binds
        want = blk + max((N / m) * outside * C, tau / kappa)
        assert abs(lse[i] - math.log(want)) < 1e-12
        np.testing.assert_allclose(out[i], (blk + (N / m) * outside) / want, atol=1e-12)     # numerator uncapped
    # every sample inside the row's block: the estimate is the lower cap tau / kappa
    one_block = np.array([order_k[0]] * 5)                          # five copies of a key of block 0
    out, lse = O.node_forward(np.zeros((N, d)), K, V, iq, ik, one_block, b, 1.0, caps=(cap_scale, kappa, T))
    for i in order_q[:b]:
        assert abs(lse[i] - math.log(b + tau / kappa)) < 1e-12


def test_row_subset_stream_is_separate_and_in_range():
    a = O.row_subset(5, 2, 3, 64, 1000)
    bb = O.sample_indices(5, 2, 3, 64, 1000)
    assert a.min() >= 0 and a.max() < 1000 and not np.array_equal(a, bb)
    x = O.philox4x32_10(np.array([[0, 2, 3, 3]], dtype=np.uint64), (5, 0))[0]
    assert a[0] == (int(x[0]) * 1000) >> 32 and a[3] == (int(x[3]) * 1000) >> 32


def test_caps_reduce_the_variance_of_the_row_sum_on_heavy_tailed_logits():
    """What the caps are for (Lemma 1's proof bounds the estimator's variance through them): with a few huge
    off-block entries the uncapped estimate of the row sum swings with whether a sample hits them; the capped one
    does not.  Heavy-tailed Q, K (Student-t, 3 d.o.f.), 400 sample sets."""
    rng = np.random.default_rng(1234)
    N, b, m, d = 256, 16, 32, 8
    Q = np.clip(rng.standard_t(3.0, (N, d)), -20, 20); K = np.clip(rng.standard_t(3.0, (N, d)), -20, 20)
    V = rng.standard_normal((N, d))
    W = O.directions(d, 4, 1)
    iq, _ = O.bucket_ids(Q, W); ik, _ = O.bucket_ids(K, W)
    T = rng.integers(0, N, m)
    l_un, l_cap = [], []
    for t in range(400):
        smp = rng.integers(0, N, m)
        l_un.append(O.node_forward(Q, K, V, iq, ik, smp, b, 0.35)[1])
        l_cap.append(O.node_forward(Q, K, V, iq, ik, smp, b, 0.35, caps=(8.0, 16.0, T))[1])
    var_un = np.var(np.array(l_un), axis=0).mean()
    var_cap = np.var(np.array(l_cap), axis=0).mean()
    print("mean variance of ln d~ over rows: uncapped", var_un, "capped", var_cap)
    assert var_cap < 0.5 * var_un


# ------------------------------------------------------------------ the alpha of Theorem 1 / Sec. 4.3
def test_alpha_closed_forms_and_explicit_loops():
    n, d = 24, 4
    rng = np.random.default_rng(3)
    K = rng.standard_normal((n, d))
    # uniform attention: every entry 1/n, a column's squared norm is 1/n, alpha = 1
    assert abs(O.alpha_diagnostic(np.zeros((n, d)), K, 1.0) - 1.0) < 1e-12
    # causal uniform attention: P_ij = 1/(i+1) for j <= i; the first column is the heaviest: n * sum_i 1/(i+1)^2
    want = n * sum(1.0 / (i + 1) ** 2 for i in range(n))
    assert abs(O.alpha_diagnostic(np.zeros((n, d)), K, 1.0, causal=True) - want) < 1e-12
    # ... and without the first 3 columns: column 3 is the heaviest of the rest
    want3 = n * sum(1.0 / (i + 1) ** 2 for i in range(3, n))
    assert abs(O.alpha_diagnostic(np.zeros((n, d)), K, 1.0, causal=True, skip_cols=3) - want3) < 1e-12
    # every query looks at one key only: that column is all ones, alpha = n^2
    Kone = np.zeros((n, d)); Kone[5, 0] = 1.0
    Qbig = np.zeros((n, d)); Qbig[:, 0] = 800.0
    assert abs(O.alpha_diagnostic(Qbig, Kone, 1.0) - n * n) < 1e-6
    # explicit loops on random inputs
    Q = rng.standard_normal((n, d))
    for causal in (False, True):
        col = [0.0] * n
        for i in range(n):
            js = [j for j in range(n) if (not causal or j <= i)]
            e = [math.exp(0.7 * float(Q[i] @ K[j])) for j in js]
            tot = sum(e)
            for j, x in zip(js, e):
                col[j] += (x / tot) ** 2
        assert abs(O.alpha_diagnostic(Q, K, 0.7, causal=causal) - n * max(col)) < 1e-10


# ------------------------------------------------------------------ sampling by value norms (Lemma 2)
def test_value_norm_weights_are_cut_squared_norms():
    rng = np.random.default_rng(4)
    from paper_2310_05869_b200 import workloads as WL
    V = WL.bf16_bits_to_f32(WL.f32_to_bf16_bits(rng.standard_normal((50, 64)).astype(np.float32)))     # bf16 values
    wq = O.value_norm_weights(V)
    exact = (V.astype(np.float64) ** 2).sum(axis=1)
    assert wq.dtype == np.uint64
    assert (np.abs(wq.astype(np.float64) / 4096.0 - exact) <= 64 * 2.0 ** -24 * exact + 1.0 / 4096.0).all()
    assert O.value_norm_weights(np.zeros((3, 8)))[0] == 0
    # coordinate order matters in fp32 and is the stated one: an explicit scalar loop gives the same integers
    for i in range(5):
        acc = np.float32(0.0)
        for c in range(64):
            acc = np.float32(acc + np.float32(V[i, c] * V[i, c]))
        assert int(wq[i]) == int(math.floor(float(acc) * 4096.0))


def test_value_norm_sampler_tiny_case_and_distribution():
    # weights 1, 0, 3: cumulative 1, 1, 4; target floor(x * 4 / 2^32) in {0, 1, 2, 3} -> index 0 for 0, index 2 otherwise
    idx, w = O.sample_by_value_norms(7, 1, 2, 4000, np.array([1, 0, 3], dtype=np.uint64))
    assert set(idx.tolist()) == {0, 2}
    assert abs((idx == 0).mean() - 0.25) < 0.03
    np.testing.assert_allclose(w[idx == 0], 4.0 / (4000 * 1.0))
    np.testing.assert_allclose(w[idx == 2], 4.0 / (4000 * 3.0))
    x = O.philox4x32_10(np.array([[0, 1, 2, 2]], dtype=np.uint64), (7, 0))[0]
    assert idx[0] == (0 if (int(x[0]) * 4) >> 32 == 0 else 2)
    # all weights zero: the uniform sampler
    i0, w0 = O.sample_by_value_norms(7, 1, 2, 16, np.zeros(10, dtype=np.uint64))
    assert (i0 == O.sample_indices(7, 1, 2, 16, 10)).all() and (w0 == 10 / 16).all()
    # chi-square against p_l = wq_l / total
    rng = np.random.default_rng(9)
    wq = rng.integers(0, 1000, 40).astype(np.uint64)
    counts = np.zeros(40)
    for seed in range(50):
        counts += np.bincount(O.sample_by_value_norms(seed, 0, 0, 2000, wq)[0], minlength=40)
    expect = 100000 * wq.astype(np.float64) / wq.sum()
    nz = expect > 0
    assert counts[~nz].sum() == 0
    chi2 = ((counts[nz] - expect[nz]) ** 2 / expect[nz]).sum()
    assert chi2 < 39 + 5 * math.sqrt(2 * 39)


def test_value_norm_sampling_is_unbiased_and_dense_form_holds():
    """E[sum_t w_t (1 - M) a_t v_t] = off-block numerator and E[sum_t w_t (1 - M) a_t] = off-block row sum
    (Lemma 2 with w = 1 / (m p)); and for one seed the implied weights reproduce the output."""
    rng = np.random.default_rng(21)
    N, b, m, d = 32, 8, 6, 4
    Q, K, _ = rand_qkv(rng, N, d)
    V = rng.standard_normal((N, d)) * rng.uniform(0.2, 3.0, (N, 1))        # rows of very different norms
    W = O.directions(d, 3, 2)
    iq, _ = O.bucket_ids(Q, W); ik, _ = O.bucket_ids(K, W)
    wq = O.value_norm_weights(V)
    _, rank_q = O.stable_argsort(iq); _, rank_k = O.stable_argsort(ik)
    M = O.sortlsh_mask(rank_q, rank_k, b)
    A = np.exp(0.5 * (Q @ K.T))
    off_sum = ((1 - M) * A).sum(axis=1)
    off_num = ((1 - M) * A) @ V
    blk_sum = (M * A).sum(axis=1)
    blk_num = (M * A) @ V
    dens, nums = [], []
    trials = 6000
    for seed in range(trials):
        smp, sw = O.sample_by_value_norms(seed, 0, 0, m, wq)
        o, l = O.node_forward(Q, K, V, iq, ik, smp, b, 0.5, sample_weights=sw)
        dens.append(np.exp(l) - blk_sum)
        nums.append(o * np.exp(l)[:, None] - blk_num)
    dens, nums = np.array(dens), np.array(nums)
    se = dens.std(axis=0) / math.sqrt(trials)
    assert (np.abs(dens.mean(axis=0) - off_sum) <= 4.5 * se + 1e-12).all()
    se = nums.std(axis=0) / math.sqrt(trials)
    assert (np.abs(nums.mean(axis=0) - off_num) <= 4.5 * se + 1e-12).all()
    for causal, n0 in ((False, 0), (True, 8)):
        o, l = O.segment_forward(Q, K, V, W, b, m, causal, n0, 5, 1, scale=0.5, value_norm_sampling=True)
        Wd = O.dense_weights(Q, K, iq, ik, b, m, 0.5, causal, n0, 5, 1, wq=wq)
        np.testing.assert_allclose(Wd.sum(axis=1), 1.0, atol=1e-12)
        np.testing.assert_allclose(Wd @ V, o, atol=1e-12)


# ------------------------------------------------------------------ directions of the node's own
def test_node_directions_streams_and_bookkeeping():
    """Node 0 is the shared set; other nodes are independent standard normals; with single-block nodes the ids do not
    matter and the recursion is still exact; with sorted nodes the result is the one rebuilt by hand from node_forward
    on the root's own ids."""
    assert np.array_equal(O.directions(16, 5, 3, node=0), O.directions(16, 5, 3))
    w1, w2 = O.directions(64, 8, 3, node=1), O.directions(64, 8, 3, node=2)
    assert not np.array_equal(w1, w2) and abs(np.corrcoef(w1.ravel(), w2.ravel())[0, 1]) < 0.15
    assert abs(w1.mean()) < 0.15 and abs(w1.std() - 1.0) < 0.15
    x = O.philox4x32_10(np.array([[0, 0, 2, 1]], dtype=np.uint64), (3, 0))[0].astype(np.float64)
    u = (x + 0.5) * 2.0 ** -32
    assert abs(float(w2.ravel()[0]) - math.sqrt(-2.0 * math.log(u[0])) * math.cos(2.0 * math.pi * u[1])) < 1e-6
    rng = np.random.default_rng(12)
    n, n0, d = 64, 8, 5
    Q, K, V = rand_qkv(rng, n, d)
    bo, bl = brute_attention(Q, K, V, 0.5, True)
    o, l = O.forward(Q[None], K[None], V[None], b=n, m=4, r=3, causal=True, n0=n0, seed=2, scale=0.5, node_directions=True)
    np.testing.assert_allclose(o[0], bo, atol=1e-11)
    # sorted nodes: the ids of level l, node j come from directions(.., node) and nothing else
    iq, ik = O.node_bucket_ids(Q, K, d, 3, 2, n0)
    L, leaf = O.causal_grid(n, n0)
    assert iq.shape == (L, n)
    W3 = O.directions(d, 3, 2, node=O.heap_node(1, 1))                 # level 1, second node: queries [48, 64), keys [32, 48)
    assert np.array_equal(iq[1, 48:64], O.bucket_ids(Q[48:64], W3)[0]) and np.array_equal(ik[1, 32:48], O.bucket_ids(K[32:48], W3)[0])
    # one level, rebuilt by hand: second-half rows merge the node's estimate (root's own ids) with exact causal attention
    n1 = 2 * n0
    o, l = O.segment_forward(Q[:n1], K[:n1], V[:n1], O.directions(d, 3, 2), 2, 5, True, n0, 2, 0, scale=0.5, node_directions=True)
    iq1, ik1 = O.node_bucket_ids(Q[:n1], K[:n1], d, 3, 2, n0)
    o21, l21 = O.node_forward(Q[n0:n1], K[:n0], V[:n0], iq1[0, n0:], ik1[0, :n0], O.sample_indices(2, 0, 0, 5, n0), 2, 0.5)
    o22, l22 = brute_attention(Q[n0:n1], K[n0:n1], V[n0:n1], 0.5, True)
    lm = np.logaddexp(l21, l22)
    np.testing.assert_allclose(l[n0:], lm, atol=1e-12)
    np.testing.assert_allclose(o[n0:], o21 * np.exp(l21 - lm)[:, None] + o22 * np.exp(l22 - lm)[:, None], atol=1e-12)
    np.testing.assert_allclose(o[:n0], brute_attention(Q[:n0], K[:n0], V[:n0], 0.5, True)[0], atol=1e-12)
    # and deeper recursions differ from the shared-directions result (the nodes below the root hash differently)
    o_nd = O.segment_forward(Q, K, V, O.directions(d, 3, 2), 4, 5, True, n0, 2, 0, scale=0.5, node_directions=True)[0]
    assert not np.allclose(o_nd, O.segment_forward(Q, K, V, O.directions(d, 3, 2), 4, 5, True, n0, 2, 0, scale=0.5)[0])
