"""CPU oracle for the HyperAttention forward pass (Han et al., arXiv 2310.05869).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, fp64 statement of what
the hot path computes.  It shares no code with the CUDA library and must never be
imported by the product path: only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it.

Every function names the passage of the paper it follows.  Where the paper is
silent the reading taken is stated in the docstring (the same readings are listed
in the design notes of the repository).

Stages (paper notation: Q, K, V are n x d; b block size; m sampled columns;
r hash bits; P_Q, P_K the sortLSH permutations; M^H the block mask):

  philox4x32_10      counter-based random words (Salmon et al., SC'11) used for
                     the hash directions and the sampled columns
  directions         r Gaussian directions of the Hamming-sorted LSH (Def. 1)
  bucket_ids         sign pattern -> Gray-ordered bucket id (Def. 1, Alg. 1 line 2)
  stable_argsort     permutations P_Q, P_K (Alg. 1 line 3)
  sortlsh_mask       the mask M^H (Alg. 1 line 4)
  query_block_size   rows per group of sorted queries when queries and keys differ in number
  causal_grid        leaves and levels of the recursive split for any sequence length
  sample_indices     l_1..l_m ~ Unif([N]) shared by all rows (Alg. 2 line 4, Sec. 4)
  row_subset         the rows T of Alg. 2 line 2 (capped variant only)
  value_norm_weights, sample_by_value_norms
                     sampling by squared row norms of V with weights 1 / (m p_l) (Lemma 2)
  exact_attention    D^-1 A V and its causal form (Sec. 1.1, Sec. 3.1)
  node_forward       block-diagonal part + sampled residual with estimated D
                     (Alg. 2 lines 7 and 9 without caps, Alg. 3, Sec. 4)
  causal_forward     recursive split (Alg. 4) carried through to outputs
  forward            all (batch, head) segments
  alpha_diagnostic   n times the largest squared column norm of the exact softmax matrix (Theorem 1, Sec. 4.3)
  dense_weights      the implied n x n row-stochastic weight matrix (tiny n only)
  dense_coefficients the matrix C with W~ = rownorm(C o exp(scale Q K^T)) (tiny n only)
  dense_backward     gradients of (out, lse) with respect to Q, K, V with the sortLSH
                     permutations and the sampled columns held fixed (tiny n only); the paper
                     times a backward pass (Sec. 4.2) but never writes it down: this is the
                     derivative of the forward map as defined above, nothing more

Parity status: every function here is pinned by the CPU tests (brute force on tiny
inputs, closed forms, the Fig. 1 example, Monte-Carlo checks, published Philox
known-answer vectors).  The spectral guarantee Eq. (1) is NOT a pin: the paper
never gives epsilon a value ("parity unpinned" for Eq. (1) only; nothing on the
hot path depends on it).
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3")
# --------------------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SHIFT32 = np.uint64(32)

DOMAIN_DIRECTIONS = 1
DOMAIN_SAMPLES = 2
DOMAIN_ROW_SUBSET = 3


def philox4x32_10(counter, key):
    """Ten rounds of Philox-4x32.  `counter` is (..., 4) and `key` is (2,) of 32-bit words.

    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 (32x32 -> 64 bit products);
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the Weyl
    constants between rounds.  Returns (..., 4) uint32.
    """
    c = np.asarray(counter, dtype=np.uint64) & _MASK32
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0 = np.uint64(int(key[0]) & 0xFFFFFFFF)
    k1 = np.uint64(int(key[1]) & 0xFFFFFFFF)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & _MASK32
            k1 = (k1 + _PHILOX_W1) & _MASK32
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SHIFT32, p0 & _MASK32
        hi1, lo1 = p1 >> _SHIFT32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def _seed_key(seed):
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return (seed & 0xFFFFFFFF, seed >> 32)


def directions(d, r, seed, node=0):
    """The r random directions of the Hamming-sorted LSH (Def. 1; Alg. 1 line 2).

    The paper cites the construction without printing it; the reading taken is r
    i.i.d. standard Gaussian directions, one set per call shared by queries, keys,
    all segments and all recursion nodes.  Entry (k, t) of W (dimension k, direction
    t) is normal number k*r + t of the stream: Philox call c (counter (c, 0, 0, 1),
    key = seed) gives words x0..x3; u_i = (x_i + 0.5) / 2^32; Box-Muller on (u0, u1)
    and on (u2, u3) gives normals 4c .. 4c+3 as (rho cos, rho sin) pairs.  The fp64
    result is rounded once to fp32 (the precision the directions are stored in).
    `node` (variant with fresh directions for every recursion node, which the paper neither
    prescribes nor excludes): the stream of node v has counter (c, 0, v, 1); node 0 is the
    shared set.
    """
    total = d * r
    calls = (total + 3) // 4
    ctr = np.zeros((calls, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(calls, dtype=np.uint64)
    ctr[:, 2] = node
    ctr[:, 3] = DOMAIN_DIRECTIONS
    x = philox4x32_10(ctr, _seed_key(seed)).astype(np.float64)
    u = (x + 0.5) * 2.0 ** -32
    z = np.empty((calls, 4), dtype=np.float64)
    for a in (0, 2):
        rho = np.sqrt(-2.0 * np.log(u[:, a]))
        ang = 2.0 * np.pi * u[:, a + 1]
        z[:, a] = rho * np.cos(ang)
        z[:, a + 1] = rho * np.sin(ang)
    return z.reshape(-1)[:total].reshape(d, r).astype(np.float32)


def sample_indices(seed, g, node, m, N):
    """l_0..l_{m-1} i.i.d. uniform on [0, N) with replacement (Alg. 2 line 4), shared by
    every query row of one (segment g, recursion node) as Sec. 4 prescribes.

    Sample j is word j & 3 of Philox call j >> 2 with counter (j >> 2, g, node, 2);
    l_j = floor(x * N / 2^32).
    """
    if m == 0:
        return np.zeros(0, dtype=np.int64)
    calls = (m + 3) // 4
    ctr = np.zeros((calls, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(calls, dtype=np.uint64)
    ctr[:, 1] = g
    ctr[:, 2] = node
    ctr[:, 3] = DOMAIN_SAMPLES
    x = philox4x32_10(ctr, _seed_key(seed)).reshape(-1)[:m].astype(np.uint64)
    return ((x * np.uint64(N)) >> _SHIFT32).astype(np.int64)


def row_subset(seed, g, node, m, n_q):
    """The rows T over which Alg. 2 line 3 takes the maximum unmasked row sum (line 2: "randomly
    choose a subset T of [n] with |T| = m"), given as POSITIONS in the sorted order of the queries
    (position p stands for row P_Q^-1(p); a uniform position is a uniform row).  Reading taken: m
    i.i.d. uniform positions (a maximum does not care about repeats), drawn like the sampled columns
    but from their own stream: counter (j >> 2, g, node, 3), word j & 3, index floor(x * n_q / 2^32)."""
    if m == 0 or n_q == 0:
        return np.zeros(0, dtype=np.int64)
    calls = (m + 3) // 4
    ctr = np.zeros((calls, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(calls, dtype=np.uint64)
    ctr[:, 1] = g
    ctr[:, 2] = node
    ctr[:, 3] = DOMAIN_ROW_SUBSET
    x = philox4x32_10(ctr, _seed_key(seed)).reshape(-1)[:m].astype(np.uint64)
    return ((x * np.uint64(n_q)) >> _SHIFT32).astype(np.int64)


VALUE_NORM_SHIFT = 12


def value_norm_weights(V):
    """Integer sampling weights floor(||V_l||^2 * 2^12) for Lemma 2's distribution p_l = ||V_l||^2 / ||V||_F^2.
    The squared norm is accumulated in fp32 in coordinate order (for bf16 values every square is exact in
    fp32, so only the additions round) and then cut to a multiple of 2^-12: integers, so that the
    cumulative sums and the sampled indices below are exactly reproducible on any machine.  (A row
    whose squared norm is below 2^-12 is never sampled.)"""
    V = np.asarray(V, dtype=np.float32)
    acc = np.zeros(V.shape[0], dtype=np.float32)
    for c in range(V.shape[1]):
        acc = (acc + V[:, c] * V[:, c]).astype(np.float32)
    return np.floor(acc.astype(np.float64) * float(1 << VALUE_NORM_SHIFT)).astype(np.uint64)


def sample_by_value_norms(seed, g, node, m, wq):
    """Lemma 2: m i.i.d. indices with probability p_l = wq_l / sum(wq) (wq from value_norm_weights, for the N
    keys of one node) and their weights 1 / (m p_l), which make sum_t w_t a_{l_t} v_{l_t} an unbiased
    estimate of sum_l a_l v_l (Lemma 2's S^T S) and sum_t w_t a_{l_t} one of the row sum.  Sample j uses
    the same Philox word x as the uniform sampler; the index is the first l whose cumulative weight
    exceeds floor(x * total / 2^32).  All weights zero: uniform sampling with weights N / m."""
    wq = np.asarray(wq, dtype=np.uint64)
    N = wq.size
    if m == 0:
        return np.zeros(0, dtype=np.int64), np.zeros(0, dtype=np.float64)
    calls = (m + 3) // 4
    ctr = np.zeros((calls, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(calls, dtype=np.uint64)
    ctr[:, 1] = g
    ctr[:, 2] = node
    ctr[:, 3] = DOMAIN_SAMPLES
    x = philox4x32_10(ctr, _seed_key(seed)).reshape(-1)[:m]
    total = int(wq.sum())
    if total == 0:
        idx = np.array([(int(v) * N) >> 32 for v in x], dtype=np.int64)
        return idx, np.full(m, N / m, dtype=np.float64)
    cum = np.cumsum(wq)
    target = np.array([(int(v) * total) >> 32 for v in x], dtype=np.uint64)
    idx = np.searchsorted(cum, target, side="right").astype(np.int64)
    return idx, total / (m * wq[idx].astype(np.float64))


# --------------------------------------------------------------------------------------
# sortLSH (Def. 1, Alg. 1)
# --------------------------------------------------------------------------------------
def gray_rank(g, r):
    """Position of sign pattern g in the reflected Gray sequence: h with h ^ (h >> 1) = g.

    Def. 1 needs adjacent bucket ids to be sign patterns at Hamming distance one
    (cyclically); ordering the patterns along the Gray sequence gives exactly that.
    """
    g = np.asarray(g, dtype=np.int64)
    h = g.copy()
    for s in range(1, r):
        h ^= g >> s
    return h


def projections(X, W):
    """<x, w_t> for every row x and direction t, in fp64."""
    return np.asarray(X, dtype=np.float64) @ np.asarray(W, dtype=np.float64)


def bucket_ids(X, W):
    """Hamming-sorted LSH bucket id of every row (Def. 1; Alg. 1 line 2).

    bit_t = [<x, w_t> > 0] (zero and negative give 0); the pattern g = sum bit_t 2^t is
    mapped to its Gray rank.  Also returns |<x, w_t>| so a caller can tell which bits
    sit too close to zero to be decided in lower precision.
    """
    p = projections(X, W)
    r = p.shape[-1]
    bits = (p > 0.0).astype(np.int64)
    g = (bits << np.arange(r, dtype=np.int64)).sum(axis=-1)
    return gray_rank(g, r).astype(np.uint8 if r <= 8 else np.int64), np.abs(p)


def stable_argsort(ids):
    """Permutation of Alg. 1 line 3.  `perm[p]` is the row placed at sorted position p;
    `rank[i]` (the paper's P(i)) is the sorted position of row i.  Equal bucket ids keep
    their original order (the paper's condition cannot hold for ties; stability makes
    the permutation unique)."""
    ids = np.asarray(ids)
    perm = np.argsort(ids, kind="stable").astype(np.int64)
    rank = np.empty_like(perm)
    rank[perm] = np.arange(perm.size, dtype=np.int64)
    return perm, rank


def query_block_size(n_q, n_k, b):
    """Rows per group of sorted queries.  Alg. 1 line 4 pairs the beta-th group of b sorted queries
    with the beta-th group of b sorted keys and is written for n_q = n_k.  Reading taken for
    n_q != n_k (cross attention, or the last off-diagonal problem of a causal sequence whose length
    the split does not divide): the key groups keep b rows and the query groups get
    b_q = ceil(b * n_q / n_k) rows, so that group beta of either side covers the same fraction of the
    sorted order; b_q = b when n_q = n_k, and ceil(n_q / b_q) <= ceil(n_k / b), so every query group
    has its key group."""
    return -((-b * n_q) // n_k)


def sortlsh_mask(rank_q, rank_k, b, b_q=None):
    """M^H_ij = 1{ floor(P_Q(i)/b_q) = floor(P_K(j)/b) }  (Alg. 1 line 4; b_q = b when the sides have
    the same number of rows, see query_block_size)."""
    bq = np.asarray(rank_q) // (b if b_q is None else b_q)
    bk = np.asarray(rank_k) // b
    return (bq[:, None] == bk[None, :]).astype(np.int64)


# --------------------------------------------------------------------------------------
# Exact attention (Sec. 1.1, Sec. 3.1): the definition, also the causal base case
# --------------------------------------------------------------------------------------
def exact_attention(Q, K, V, scale, causal=False, rows=None):
    """Att = D^-1 A V with A = exp(scale * Q K^T); causal keeps entries i >= j
    (M^C_ij = 1{i >= j}, diagonal included).  Returns (out, lse) with lse = ln D_ii.
    `rows` restricts the evaluation to some query rows (rows are independent)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    idx = np.arange(Q.shape[0]) if rows is None else np.asarray(rows, dtype=np.int64)
    s = scale * (Q[idx] @ K.T)
    if causal:
        s = np.where(idx[:, None] >= np.arange(K.shape[0])[None, :], s, -np.inf)
    mx = s.max(axis=1, keepdims=True)
    a = np.exp(s - mx)
    den = a.sum(axis=1, keepdims=True)
    out = (a @ V) / den
    lse = (mx + np.log(den))[:, 0]
    return out, lse


def alpha_diagnostic(Q, K, scale, causal=False, skip_cols=0):
    """alpha = n * max_j ||D^-1 A e_j||_2^2 (Theorem 1; Sec. 4.3): n times the largest squared column
    norm of the exact softmax matrix, the first skip_cols columns left out of the maximum."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    n = Q.shape[0]
    s = scale * (Q @ K.T)
    if causal:
        s = np.where(np.arange(n)[:, None] >= np.arange(K.shape[0])[None, :], s, -np.inf)
    P = np.exp(s - s.max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    return n * float((P * P).sum(axis=0)[skip_cols:].max())


# --------------------------------------------------------------------------------------
# One non-causal HyperAttention problem (Alg. 1-3 as specialised in Sec. 4)
# --------------------------------------------------------------------------------------
def unmasked_row_sum_bound(Q, K, rank_q, rank_k, T, b, b_q, scale):
    """ln tau of Alg. 2 line 3: tau = max over j in T of <1 - M^H_j, exp(K q_j)>, the largest
    row sum of the entries outside the mask among the rows of T (minus infinity if T is empty or
    every row of T has all its keys inside its block)."""
    ltau = -np.inf
    for j in np.asarray(T, dtype=np.int64):
        s = scale * (K @ Q[j])
        s = s[(rank_k // b) != (rank_q[j] // b_q)]
        if s.size:
            mx = s.max()
            ltau = max(ltau, mx + math.log(np.exp(s - mx).sum()))
    return ltau


def node_forward(Q, K, V, ids_q, ids_k, samples, b, scale, rows=None, caps=None, sample_weights=None):
    """HyperAttention on n_q queries x N keys (n_q = N in the paper; see query_block_size for the
    grouping when they differ).

    For query row i in sorted block beta = floor(P_Q(i)/b_q):
      * masked part: the keys j with floor(P_K(j)/b) = beta, exact exp(s_ij)
        (Alg. 2, "row-sum of masked entries"; Sec. 4 block-diagonal product);
      * residual: (N/m) * sum over samples l_t with M^H_{i,l_t} = 0 of exp(s_{i,l_t})
        (Alg. 2 line 7 without the cap C_i; collisions get weight zero, duplicates
        count with their multiplicity);
      * d~_i = masked + residual (Alg. 2 line 9 without the lower cap);
      * numerator: same weights times the value rows (sampled indices reused for the
        approximate matrix product, Sec. 4; uniform p = 1/N in Lemma 2 gives weight N/m).
    out_i = numerator_i / d~_i, lse_i = ln d~_i.  If b >= N the whole problem is one
    block and nothing is sampled.  Returns (out, lse) for `rows` (default all rows),
    in original row order.

    caps = (cap_scale, kappa, T) switches on the caps of Alg. 2 (lines 3, 6, 7 and 9 as printed; T holds
    positions of the sorted query order, see row_subset):
      tau   = max_{j in T} <1 - M^H_j, exp(K q_j)>                                  (line 3)
      C_i   = cap_scale * m / (N ln N) * (masked_i + tau / kappa)                   (line 6; the paper
              writes Theta(eps^2 m / (n log n) (...)): the constant times eps^2 is the caller's cap_scale)
      d_i   = (N/m) sum_t (1 - M^H_{i,l_t}) min(exp(s_{i,l_t}), C_i)                (line 7)
      d~_i  = masked_i + max(d_i, tau / kappa)                                      (line 9)
    The numerator is unchanged (Alg. 3 multiplies D~^-1 by the sampled product A V; the caps belong
    to the row-sum estimate of Alg. 2 only), so with caps the outputs are no longer convex
    combinations of value rows.  cap_scale = inf and kappa = inf switch both caps off.

    sample_weights (one per sample) replaces the uniform weight N/m: with samples drawn from another
    distribution p the weight of sample t is 1 / (m p_{l_t}) (Lemma 2; sample_by_value_norms), in
    the numerator and in the row sum alike.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N = K.shape[0]
    n_q = Q.shape[0]
    if b >= N:
        return exact_attention(Q, K, V, scale, causal=False, rows=rows)
    b_q = query_block_size(n_q, N, b)
    # N need not be a multiple of b: Alg. 1 line 4 defines the mask through floor(P(i)/b), so the
    # last sorted block simply has N mod b rows of Q and of K (the slices below end at N)
    perm_q, rank_q = stable_argsort(ids_q)
    perm_k, rank_k = stable_argsort(ids_k)
    samples = np.asarray(samples, dtype=np.int64)
    m = samples.size
    want = np.arange(n_q) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((want.size, V.shape[1]), dtype=np.float64)
    lse = np.zeros(want.size, dtype=np.float64)
    blk_of_want = rank_q[want] // b_q
    Ks, Vs = K[samples], V[samples]
    blk_of_sample = rank_k[samples] // b
    capped = caps is not None and m > 0
    if capped:
        cap_scale, kappa, T = caps                                       # T: positions in the sorted query order
        lfloor = unmasked_row_sum_bound(Q, K, rank_q, rank_k, perm_q[np.asarray(T, dtype=np.int64)], b, b_q, scale) - math.log(kappa)   # ln(tau / kappa)
        coef = cap_scale * m / (N * math.log(N))
    for beta in np.unique(blk_of_want):
        sel = np.nonzero(blk_of_want == beta)[0]
        qi = want[sel]
        J = perm_k[beta * b:(beta + 1) * b]
        s_blk = scale * (Q[qi] @ K[J].T)
        mx = s_blk.max(axis=1, keepdims=True)
        if m > 0:
            keep = (blk_of_sample != beta).astype(np.float64)          # 1 - M^H_{i, l_t}
            s_smp = scale * (Q[qi] @ Ks.T)
            if keep.any():
                mx = np.maximum(mx, s_smp[:, keep > 0].max(axis=1, keepdims=True))
            if capped and lfloor > -np.inf:
                mx = np.maximum(mx, lfloor)
            if sample_weights is None:
                w = (N / m) * keep[None, :] * np.exp(np.where(keep[None, :] > 0, s_smp - mx, -np.inf))
            else:
                sw = np.asarray(sample_weights, dtype=np.float64)
                w = sw[None, :] * keep[None, :] * np.exp(np.where(keep[None, :] > 0, s_smp - mx, -np.inf))
        a = np.exp(s_blk - mx)
        den = a.sum(axis=1, keepdims=True)
        num = a @ V[J]
        if m > 0:
            num = num + w @ Vs
            # Alg. 2 line 7: d_i = (N/m) sum_t (1 - M) min(exp(s), C_i); line 9: d~_i = masked + max(d_i, tau / kappa)
            # (without caps C_i is infinite and tau / kappa is zero)
            floor = np.exp(lfloor - mx) if capped else 0.0               # tau / kappa in units of exp(mx)
            cap = coef * (den + floor) if capped else np.inf             # C_i
            p = np.exp(np.where(keep[None, :] > 0, s_smp - mx, -np.inf))
            if sample_weights is None:
                d_i = (N / m) * (keep[None, :] * np.minimum(p, cap)).sum(axis=1, keepdims=True)
            else:
                d_i = (sw[None, :] * keep[None, :] * np.minimum(p, cap)).sum(axis=1, keepdims=True)
            den = den + np.maximum(d_i, floor)
        out[sel] = num / den
        lse[sel] = (mx + np.log(den))[:, 0]
    return out, lse


# --------------------------------------------------------------------------------------
# Causal masking by recursion (Alg. 4, Fig. 2), carried through to the outputs
# --------------------------------------------------------------------------------------
def causal_grid(n, n0):
    """(L, leaf): Alg. 4 halves the sequence until a part is not longer than n0.  L halvings give
    2^L leaves of leaf = ceil(n / 2^L) rows.  Reading taken when 2^L does not divide n (Alg. 4 line 2
    only speaks of equal halves): the split points are those of the length rounded up to leaf * 2^L,
    i.e. every part is cut at half of its nominal length and the rows that the rounded-up length
    would have beyond n do not exist - the last leaf is short, and so is the query side of the last
    off-diagonal problem of a level (queries and keys then differ in number, see query_block_size)."""
    L = 0
    while -((-n) >> L) > n0:
        L += 1
    return L, -((-n) >> L)


def draw_samples(seed, g, node, m, N, wq=None):
    """(indices, weights or None): uniform (Sec. 4) or, given the keys' integer weights, by value norms (Lemma 2)."""
    if wq is None:
        return sample_indices(seed, g, node, m, N), None
    return sample_by_value_norms(seed, g, node, m, wq)


def node_bucket_ids(Q, K, d, r, seed, n0):
    """Bucket ids when every recursion node of a causal call hashes with directions of its own
    (directions(.., node=v)): two (L, n) arrays; entry (l, i) of the first is the id of query row i
    in the level-l node whose second half holds it, entry (l, i) of the second the id of key row i in
    the level-l node whose first half holds it (a row is on one side of exactly one node per level;
    the other entries are left at zero)."""
    n = Q.shape[0]
    L, leaf = causal_grid(n, n0)
    iq = np.zeros((L, n), dtype=np.uint8)
    ik = np.zeros((L, n), dtype=np.uint8)
    for level in range(L):
        s = leaf << (L - 1 - level)
        for j in range(1 << level):
            q0, k0 = (2 * j + 1) * s, 2 * j * s
            e = min(q0 + s, n)
            if e <= q0:
                continue
            W = directions(d, r, seed, node=heap_node(level, j))
            iq[level, q0:e] = bucket_ids(Q[q0:e], W)[0]
            ik[level, k0:k0 + s] = bucket_ids(K[k0:k0 + s], W)[0]
    return iq, ik


def causal_forward(Q, K, V, ids_q, ids_k, b, m, scale, n0, seed, g, rows=None, caps=None, wq=None):
    """Causal HyperAttention.  A part that is a single leaf gets exact causal attention (the paper
    recurses until the length falls below a base size and uses an exact kernel there).  A larger
    part of nominal length S is split at S/2 (Alg. 4 line 2); the two halves recurse (line 3); the
    non-causal algorithm runs on (Q2, K1, V1) (line 4); rows of the second half add the two row
    sums, D~_21 + D~_C22 (line 5), and so their outputs combine with weights proportional to the
    two estimated row sums ("merging attention outputs", Sec. 4.2).  Recursion nodes are numbered
    like a binary heap (root 0, children 2v+1 and 2v+2) and the off-diagonal problem of node v
    draws its samples from stream (g, v).  See causal_grid for lengths that the split does not
    divide."""
    n = Q.shape[0]
    L, leaf = causal_grid(n, n0)
    want = np.arange(n) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((want.size, V.shape[1]), dtype=np.float64)
    lse = np.zeros(want.size, dtype=np.float64)
    ids_q, ids_k = np.asarray(ids_q), np.asarray(ids_k)
    per_level = ids_q.ndim == 2                       # (L, n): ids from directions of the node's own (node_bucket_ids)

    def part(a, S, node, sel):
        """rows want[sel] (all inside [a, a + S)) of the causal problem on rows [a, min(a + S, n))"""
        if sel.size == 0:
            return
        e = min(a + S, n)
        if S == leaf:
            o, l = exact_attention(Q[a:e], K[a:e], V[a:e], scale, causal=True, rows=want[sel] - a)
            out[sel], lse[sel] = o, l
            return
        h = S // 2
        first = sel[want[sel] < a + h]
        second = sel[want[sel] >= a + h]
        part(a, h, 2 * node + 1, first)
        if second.size:
            part(a + h, h, 2 * node + 2, second)
            r2 = want[second] - (a + h)
            mm = m if b < h else 0
            smp, sw = draw_samples(seed, g, node, mm, h, None if wq is None else wq[a:a + h])
            nc = None if caps is None else (caps[0], caps[1], row_subset(seed, g, node, mm, e - (a + h)))
            level = (node + 1).bit_length() - 1
            iq = ids_q[level, a + h:e] if per_level else ids_q[a + h:e]
            ik = ids_k[level, a:a + h] if per_level else ids_k[a:a + h]
            o21, l21 = node_forward(Q[a + h:e], K[a:a + h], V[a:a + h], iq, ik, smp, b, scale, rows=r2, caps=nc,
                                    sample_weights=sw)
            o22, l22 = out[second].copy(), lse[second].copy()
            l = np.logaddexp(l21, l22)
            out[second] = o21 * np.exp(l21 - l)[:, None] + o22 * np.exp(l22 - l)[:, None]
            lse[second] = l

    part(0, leaf << L, 0, np.arange(want.size))
    return out, lse


def heap_node(level, j):
    """Heap index of the j-th recursion node of a level (root is level 0)."""
    return (1 << level) - 1 + j


# --------------------------------------------------------------------------------------
# Whole forward pass
# --------------------------------------------------------------------------------------
def segment_forward(Q, K, V, W, b, m, causal, n0, seed, g, scale=None, rows=None,
                    ids_q=None, ids_k=None, caps=None, value_norm_sampling=False, node_directions=False):
    """Forward pass of one (batch, head) segment.  `ids_q` / `ids_k` may be injected
    (e.g. the bucket ids another implementation produced) so that later stages can be
    compared even when a sign bit at |projection| ~ 0 was decided differently.
    caps = (cap_scale, kappa) runs Alg. 2 with its caps (see node_forward); every off-diagonal
    problem then draws its own row subset T.  value_norm_sampling draws the sampled columns by
    squared row norms of V (Lemma 2) instead of uniformly (Sec. 4).  node_directions (causal calls
    with at least one level): every recursion node hashes with directions of its own, and injected
    ids are (L, n) arrays as node_bucket_ids returns them."""
    Q = np.asarray(Q, dtype=np.float64)
    n, d = Q.shape
    n_k = np.asarray(K).shape[0]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    if node_directions and causal and causal_grid(n, n0)[0] > 0:
        if ids_q is None or ids_k is None:
            r = np.asarray(W).shape[1]
            ids_q, ids_k = node_bucket_ids(Q, np.asarray(K, dtype=np.float64), d, r, seed, n0)
    else:
        if ids_q is None:
            ids_q, _ = bucket_ids(Q, W)
        if ids_k is None:
            ids_k, _ = bucket_ids(K, W)
    wq = value_norm_weights(V) if value_norm_sampling else None
    if causal:
        assert n_k == n, "the causal mask is defined for a square attention matrix"
        return causal_forward(Q, K, V, ids_q, ids_k, b, m, scale, n0, seed, g, rows=rows, caps=caps, wq=wq)
    mm = m if b < n_k else 0
    smp, sw = draw_samples(seed, g, 0, mm, n_k, wq)
    nc = None if caps is None else (caps[0], caps[1], row_subset(seed, g, 0, mm, n))
    return node_forward(Q, K, V, ids_q, ids_k, smp, b, scale, rows=rows, caps=nc, sample_weights=sw)


def forward(Q, K, V, b, m, r, causal=False, n0=0, seed=0, scale=None, caps=None, value_norm_sampling=False,
            node_directions=False):
    """Q: (G, n, d); K, V: (G, n_k, d).  Returns out (G, n, d) and lse (G, n), fp64."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    G, n, d = Q.shape
    W = directions(d, r, seed)
    out = np.zeros((G, n, d), dtype=np.float64)
    lse = np.zeros((G, n), dtype=np.float64)
    for g in range(G):
        out[g], lse[g] = segment_forward(Q[g], K[g], V[g], W, b, m, causal, n0, seed, g, scale, caps=caps,
                                         value_norm_sampling=value_norm_sampling, node_directions=node_directions)
    return out, lse


# --------------------------------------------------------------------------------------
# Dense cross-form (tiny n only): the n x n weight matrix the method implies
# --------------------------------------------------------------------------------------
def _dense_unnormalised(Q, K, ids_q, ids_k, samples, b, scale):
    """(M^H + (N/m) c_j (1 - M^H)) o exp(scale Q K^T), c_j = multiplicity of key j among
    the samples (Alg. 2 lines 7 and 9 without caps, written as one matrix)."""
    N = K.shape[0]
    A = np.exp(scale * (np.asarray(Q, np.float64) @ np.asarray(K, np.float64).T))
    if b >= N:
        return A
    _, rank_q = stable_argsort(ids_q)
    _, rank_k = stable_argsort(ids_k)
    M = sortlsh_mask(rank_q, rank_k, b, query_block_size(np.asarray(Q).shape[0], N, b)).astype(np.float64)
    c = np.bincount(np.asarray(samples, dtype=np.int64), minlength=N).astype(np.float64)
    m = max(len(samples), 1)
    return (M + (N / m) * c[None, :] * (1.0 - M)) * A


def dense_weights(Q, K, ids_q, ids_k, b, m, scale, causal, n0, seed, g, wq=None):
    """Row-normalised weights W~ (n x n_k) with out = W~ V; causal problems are assembled quadrant by
    quadrant exactly as Fig. 2 / Alg. 4 split the matrix (causal_grid for the split points)."""
    C = dense_coefficients(np.asarray(Q).shape[0], ids_q, ids_k, b, m, causal, n0, seed, g, n_k=np.asarray(K).shape[0], wq=wq)
    U = C * np.exp(scale * (np.asarray(Q, np.float64) @ np.asarray(K, np.float64).T))
    return U / U.sum(axis=1, keepdims=True)


# --------------------------------------------------------------------------------------
# Backward pass (tiny n only): derivative of the forward map, discrete choices held fixed
# --------------------------------------------------------------------------------------
def dense_coefficients(n, ids_q, ids_k, b, m, causal, n0, seed, g, n_k=None, wq=None):
    """C (n x n_k, entries >= 0) such that the forward pass is out = rownorm(C o A) V,
    lse = ln rowsum(C o A), A = exp(scale Q K^T).  C depends on Q and K only through the
    bucket ids: C_ij = 1 on the block mask M^H, (N/m) * multiplicity of j among the
    samples elsewhere (Alg. 2 lines 7 and 9 without caps), the lower triangle of ones in
    an exact causal leaf, zero above the diagonal blocks of the recursion (Alg. 4).  wq: the keys'
    integer weights when the columns are sampled by value norms (then the coefficient of a sampled key
    is the sum of the weights 1 / (m p) of the samples that hit it)."""
    ids_q, ids_k = np.asarray(ids_q), np.asarray(ids_k)
    n_k = n if n_k is None else n_k

    def block(iq, ik, node, wq_node=None):
        N = ik.shape[0]
        if b >= N:
            return np.ones((iq.shape[0], N))
        _, rank_q = stable_argsort(iq)
        _, rank_k = stable_argsort(ik)
        M = sortlsh_mask(rank_q, rank_k, b, query_block_size(iq.shape[0], N, b)).astype(np.float64)
        smp, sw = draw_samples(seed, g, node, m, N, wq_node)
        if sw is None:
            c = (N / max(m, 1)) * np.bincount(np.asarray(smp, dtype=np.int64), minlength=N).astype(np.float64)
        else:
            c = np.bincount(np.asarray(smp, dtype=np.int64), weights=sw, minlength=N)       # sum of the weights of the samples that hit a key
        return M + c[None, :] * (1.0 - M)

    if not causal:
        return block(ids_q, ids_k, 0, wq)
    assert n_k == n
    L, leaf = causal_grid(n, n0)
    C = np.zeros((n, n))

    def part(a, S, node):
        e = min(a + S, n)
        if e <= a:
            return
        if S == leaf:
            C[a:e, a:e] = np.tril(np.ones((e - a, e - a)))
            return
        h = S // 2
        part(a, h, 2 * node + 1)
        part(a + h, h, 2 * node + 2)
        if e > a + h:
            C[a + h:e, a:a + h] = block(ids_q[a + h:e], ids_k[a:a + h], node, None if wq is None else wq[a:a + h])

    part(0, leaf << L, 0)
    return C


def dense_backward(Q, K, V, C, scale, d_out, d_lse=None, with_term_sizes=False):
    """Gradients of L = <d_out, out> + <d_lse, lse> for out = P V, P = rownorm(C o A),
    lse = ln rowsum(C o A), A = exp(scale Q K^T), C constant:
        dV = P^T d_out
        dP = d_out V^T
        dS = P o (dP - rowsum(P o dP) + d_lse)      (softmax Jacobian; d lse_i / d s_ij = P_ij)
        dQ = scale dS K,   dK = scale dS^T Q.
    Returns (dQ, dK, dV), fp64; with_term_sizes adds, per gradient, the sum of the absolute
    values of the terms behind every entry (a yardstick for rounding errors)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    d_out = np.asarray(d_out, dtype=np.float64)
    s = scale * (Q @ K.T)
    with np.errstate(divide="ignore"):
        z = s + np.log(C)
    z = z - z.max(axis=1, keepdims=True)
    P = np.exp(z)
    P = P / P.sum(axis=1, keepdims=True)
    dV = P.T @ d_out
    dP = d_out @ V.T
    inner = (P * dP).sum(axis=1, keepdims=True)
    dS = P * (dP - inner)
    if d_lse is not None:
        dS = dS + P * np.asarray(d_lse, dtype=np.float64)[:, None]
    grads = (scale * (dS @ K), scale * (dS.T @ Q), dV)
    if not with_term_sizes:
        return grads
    # sums of the absolute values of the terms each gradient entry is made of (what a rounding of
    # every term by a relative eps can move it by, divided by eps): the two products inside dS
    # count separately
    # (delta_i = <dO_i, O_i> counts with the absolute values of ITS terms: a caller that forms it
    # from a rounded O moves it by eps times that sum, however much the terms cancel)
    delta_terms = (np.abs(d_out) * np.abs(P @ V)).sum(axis=1, keepdims=True)
    T = P * (np.abs(dP) + np.abs(inner) + delta_terms)
    sizes = (scale * (T @ np.abs(K)), scale * (T.T @ np.abs(Q)), P.T @ np.abs(d_out))
    return grads, sizes
