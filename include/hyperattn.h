/*
 * hyperattn.h -- C ABI of the B200 (sm_100a) HyperAttention forward library.
 *
 * Method: Han, Jayaram, Karbasi, Mirrokni, Woodruff, Zandieh, "HyperAttention:
 * Long-context Attention in Near-Linear Time" (arXiv 2310.05869).  The library
 * computes the practical forward pass of Sec. 4 ("Implementation Detail"):
 *
 *   1. sortLSH (Def. 1, Alg. 1): every query and key row is hashed by the signs of
 *      r = hash_bits Gaussian projections, the sign pattern is mapped to its position
 *      in the reflected Gray sequence (adjacent bucket ids differ in one sign), and
 *      queries and keys are argsorted (stably) by bucket id.
 *   2. Exact softmax attention inside the b x b diagonal blocks of the sorted order
 *      (the mask M^H of Alg. 1 line 4; Sec. 4).
 *   3. Residual (Alg. 2 lines 4, 7 and 9 without the caps; Alg. 3; Sec. 4): m key
 *      indices drawn i.i.d. uniformly, shared by all query rows; sampled entries outside
 *      a row's block enter the row sum and the numerator with weight N/m.
 *   4. out_i = numerator_i / d~_i, lse_i = ln d~_i.  With causal masking the recursive
 *      split of Alg. 4 / Fig. 2 is applied: the two diagonal halves recurse down to an
 *      exact causal base case of n0 rows, the lower-left quadrant is a non-causal
 *      HyperAttention problem, and the row sums (hence the outputs) of the second half
 *      are combined (Alg. 4 line 5).
 *
 * Conventions common to all entry points
 *   - q, k, v, out are DEVICE pointers to contiguous [B, H, n, d] tensors, d fastest;
 *     lse is a DEVICE pointer to [B, H, n] floats (natural logarithm of the estimated
 *     row sum d~_i of exp(softmax_scale * <q_i, k_j>)).  All must be 16-byte aligned.
 *   - The caller owns every buffer passed in; the library neither frees nor keeps them.
 *     `out`/`lse` must not alias an input.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All work
 *     is enqueued on it; no entry point synchronises unless it says so.
 *   - Return value: 0 on success, a negative hyperattn_status otherwise.  On a
 *     host-detected error nothing is launched and no output is written.
 *   - Shapes: d in {64, 128}; 1 <= hash_bits <= 8; samples >= 0; block >= 1.
 *     block need not divide n (or a recursion node's size): the mask of Alg. 1 line 4 is
 *     floor(P(i) / block), so the last sorted block is short; block >= n makes the problem one
 *     exact block.  Causal: Alg. 4 halves the rows until a part is not longer than n0 (L
 *     halvings, 2^L exact causal leaves of leaf = ceil(n / 2^L) rows; L = 0 if n <= n0).  Any n
 *     is accepted: every part is cut at half of its nominal length leaf * 2^k, and when 2^L
 *     does not divide n the rows beyond n simply do not exist, so the last leaf is short and
 *     the last off-diagonal problem of a level has fewer queries than keys (it is then grouped
 *     like a call with n != n_k, see hyperattn_params.n_k).  n = 100003 with n0 = 4096 has 32
 *     leaves of 3126 rows, the last one of 3097.
 *   - Recursion nodes are numbered like a binary heap: the off-diagonal problem of the
 *     j-th node of level l (root level 0) is node (2^l - 1) + j; it pairs query rows
 *     [(2j+1)s, (2j+2)s) with key rows [2js, (2j+1)s), s = leaf * 2^(L-1-l)
 *     (= n / 2^(l+1) when 2^L divides n; query rows beyond n do not exist).  A non-causal
 *     call has the single node 0 over all rows.
 *   - Random numbers: Philox4x32-10 keyed by `seed`; directions use counter
 *     (c, 0, 0, 1), samples of (segment g, node v) use counter (j >> 2, g, v, 2),
 *     word j & 3, index = floor(word * N / 2^32).
 */
#ifndef HYPERATTN_H_
#define HYPERATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum hyperattn_status {
  HYPERATTN_OK = 0,
  HYPERATTN_INVALID_ARGUMENT = -1,   /* null pointer, non-positive size, bad enum */
  HYPERATTN_UNSUPPORTED_SHAPE = -2,  /* shape rules above violated */
  HYPERATTN_MISALIGNED = -3,         /* a pointer is not 16-byte aligned, or out aliases an input */
  HYPERATTN_WORKSPACE_TOO_SMALL = -4,
  HYPERATTN_CUDA_ERROR = -5,         /* a CUDA runtime call failed */
  HYPERATTN_DEVICE_TIMEOUT = -6      /* a bounded device-side wait gave up (status word) */
} hyperattn_status;

typedef enum hyperattn_dtype {
  HYPERATTN_BF16 = 0,
  HYPERATTN_FP32 = 1
} hyperattn_dtype;

/* Optional device buffers that receive the intermediate results of the integer stages
 * (needed to compare them bit for bit with a reference).  Any member may be NULL.
 * Let G = B*H, LV = number of levels (1 if non-causal or n <= n0, else L),
 * NL = rows per (level, segment, side): max(n, n_k) if non-causal, leaf * 2^(L-1) if causal with
 * L >= 1 (n/2 when 2^L divides n; entries of rows that do not exist are left untouched),
 * NODES = 1 if non-causal, 2^L - 1 if causal (0 if n <= n0).
 *   q_ids        : uint8 [G, n]        bucket id of every query row (Def. 1)
 *   k_ids        : uint8 [G, n_k]      bucket id of every key row
 *   perm_q,perm_k: int32 [LV, G, NL]   node j of level l occupies [j*s, (j+1)*s);
 *                                      entry p = row (relative to the node's first query /
 *                                      key row) placed at sorted position p (Alg. 1 line 3)
 *   rank_k       : int32 [LV, G, NL]   inverse of perm_k (the paper's P_K)
 *   samples      : int32 [G, NODES, m] sampled key indices relative to the node (Alg. 2 line 4)
 *   near_zero_bits: one uint64 counter, incremented by the number of hash bits whose
 *                   projection magnitude is below 1e-4 (caller zeroes it) */
typedef struct hyperattn_debug {
  uint8_t* q_ids;
  uint8_t* k_ids;
  int32_t* perm_q;
  int32_t* perm_k;
  int32_t* rank_k;
  int32_t* samples;
  unsigned long long* near_zero_bits;
  /* capped calls only (hyperattn_params.capped): */
  int32_t* row_subset;   /* int32 [G, NODES, m]: the probe rows T of Alg. 2 line 2, as positions in the node's
                            sorted query order */
  float* log2_tau;       /* float [G, NODES]: log2 of tau (Alg. 2 line 3) with the softmax scale applied, i.e.
                            ln(tau) / ln 2; minus infinity for a node without probe rows or unmasked entries */
  /* sampling by value norms only (hyperattn_params.sampling): */
  float* sample_log2w;   /* float [G, NODES, m]: log2 of the weight 1 / (m p_l) of every drawn column */
} hyperattn_debug;

typedef struct hyperattn_params {
  const void* q;
  const void* k;
  const void* v;
  void* out;             /* [B,H,n,d] in out_dtype */
  float* lse;            /* [B,H,n] */
  int B, H, n, d;
  int block;             /* b of Alg. 1 */
  int samples;           /* m of Alg. 2 */
  int hash_bits;         /* r of Def. 1 */
  int causal;            /* 0 / 1 */
  int n0;                /* exact causal base size (ignored if !causal) */
  uint64_t seed;
  int dtype;             /* hyperattn_dtype of q, k, v */
  int out_dtype;         /* hyperattn_dtype of out (fp32 out with bf16 inputs is allowed) */
  float softmax_scale;   /* <= 0 selects 1/sqrt(d) */
  void* workspace;       /* device scratch owned by the caller, or NULL: the library then
                            uses a private per-device buffer that it grows on demand (the
                            growing call synchronises the device, frees the old buffer and
                            allocates a new one) and keeps until hyperattn_release(); calls
                            that share it must not overlap.  Stream capture: a call made while
                            `stream` is being captured never allocates or synchronises; it
                            returns HYPERATTN_WORKSPACE_TOO_SMALL if it has no caller's workspace
                            and the private one is missing or too small.  A captured graph holds
                            the workspace's address: capture with a caller-owned workspace, or
                            know that a graph captured on the private buffer is invalidated by
                            any later call that grows it and by hyperattn_release(). */
  size_t workspace_bytes;
  const hyperattn_debug* debug; /* may be NULL */
  void* stream;
  /* ---- options added after version 1; all-zero selects the behaviour described above ---- */
  int precise;           /* 1: every softmax weight enters the weights-times-values product as a pair of
                            bf16 numbers (relative error 2^-17 instead of 2^-9).  With single bf16 weights an
                            output entry can be off by 2^-8 max|v|, which is 2e-2 for values of N(0,1) size
                            but more for heavy-tailed values; this mode keeps the error below 2e-2 for values
                            up to +-20 at the price of twice the weights-times-values products.  bf16 inputs only. */
  int n_k;               /* rows of k and v per (batch, head): k, v are [B, H, n_k, d]; 0 means n.  Non-causal
                            calls only (the causal mask is defined for a square matrix).  Alg. 1 line 4 pairs the
                            beta-th group of sorted queries with the beta-th group of sorted keys and is written
                            for n = n_k; with n != n_k the key groups keep `block` rows and the query groups get
                            ceil(block * n / n_k) rows, so that a group of either side covers the same fraction of
                            its sorted order (every query group has a key group).  The samples are drawn from the
                            n_k keys and weigh n_k / samples. */
  int capped;            /* 1: the row-sum estimate of every sorted node carries the caps of Alg. 2 as printed:
                              tau  = max over a random set T of m probe rows of the row sum outside the mask (line 3;
                                     T = m i.i.d. uniform positions of the node's sorted query order, Philox counter
                                     (j >> 2, g, v, 3)),
                              C_i  = cap_scale * m / (N ln N) * (masked_i + tau / kappa)          (line 6),
                              d_i  = (N/m) sum_t (1 - M_{i,l_t}) min(exp(s_{i,l_t}), C_i)         (line 7),
                              d~_i = masked_i + max(d_i, tau / kappa)                             (line 9),
                            masked_i the exact row sum inside the block.  The numerator keeps the uncapped sampled
                            weights (Alg. 3), so out_i = numerator_i / d~_i is no longer a convex combination of
                            value rows.  The paper gives the constant of line 6 only as Theta(eps^2 ...): the caller
                            supplies it.  Costs one extra pass of m rows against all keys of every node.  bf16
                            inputs, forward only, not together with `precise`. */
  float cap_scale;       /* the constant (times eps^2) of Alg. 2 line 6; > 0 when capped */
  float kappa;           /* kappa of Alg. 2; > 0 when capped */
  int sampling;          /* hyperattn_sampling: how the m residual columns of a sorted node are drawn.
                            HYPERATTN_SAMPLE_UNIFORM (Sec. 4): uniformly, weight N/m each.
                            HYPERATTN_SAMPLE_VALUE_NORMS (Lemma 2): key l with probability p_l proportional to
                            ||V_l||^2 over the node's keys, weight 1 / (m p_l) in the numerator and in the row sum.
                            The distribution is made of integers so that the indices are reproducible: the squared
                            norm is accumulated in fp32 in coordinate order and cut to a multiple of 2^-12; draw j is
                            the first key whose cumulative weight exceeds floor(x * total / 2^32), x the Philox word
                            of the uniform sampler (counter (j >> 2, g, v, 2), word j & 3); all weights zero falls
                            back to uniform.  Costs one more pass over V.  bf16 inputs, forward only, samples <= 512,
                            not together with `precise` or `capped`. */
  int node_directions;   /* 1 (causal calls): every recursion node hashes its queries and keys with directions of its own
                            (Philox counter (c, 0, v, 1) for node v; node 0 is the shared set) instead of one set per
                            call.  The paper is silent on this; one shared set is the default.  Every row is then hashed
                            once per level, and the exported bucket ids are [LV, G, n]: entry (l, g, i) of q_ids is the id
                            of query row i in the level-l node whose second half holds it, of k_ids the id of key row i in
                            the level-l node whose first half holds it (other entries are not written).  Forward only, at
                            most 4095 nodes. */
} hyperattn_params;

typedef enum hyperattn_sampling {
  HYPERATTN_SAMPLE_UNIFORM = 0,
  HYPERATTN_SAMPLE_VALUE_NORMS = 1
} hyperattn_sampling;

/* HyperAttention forward (Alg. 1-4 as specialised in Sec. 4) with bf16 inputs and
 * output, softmax scale 1/sqrt(d) and the library's private workspace. */
int hyperattn_forward(const void* q, const void* k, const void* v, void* out, float* lse,
                      int B, int H, int n, int d, int block, int samples, int hash_bits,
                      int causal, int n0, uint64_t seed, void* stream);

/* The same computation with every option explicit. */
int hyperattn_forward_ex(const hyperattn_params* p);

/* The same computation for HOST buffers: q, k, v, out, lse of *p are host pointers (pinned
 * memory makes the copies asynchronous).  The (batch, head) segments are independent, so they
 * go through a private device staging area in up to sixteen groups: the copy of the next group to
 * the device and the copy of the previous group's out / lse back run on two streams of the
 * library while a group is computed on `stream`.  Everything is ordered after the work already
 * queued on `stream`, and `stream` is made to wait for the last copy back: the caller
 * synchronises `stream` before reading the results.  Results are bit-identical to
 * hyperattn_forward_ex on device copies of the same tensors.  With debug outputs requested the
 * batch is one group.  The staging area is grown on demand (that call synchronises the device)
 * and kept, like the two streams, until hyperattn_release().  Calls on one device share the staging
 * area, the two streams and their events: they must not overlap (issue them from one thread, or
 * order them yourself). */
int hyperattn_forward_host(const hyperattn_params* p);

/* Backward pass.  The paper times a backward pass (Sec. 4.2) without writing it down; this is the
 * derivative of the forward map of Alg. 2-4 as computed by hyperattn_forward_ex, with the sortLSH
 * permutations and the sampled columns held fixed (they are recomputed from q, k and the seed, so
 * *p must be the forward call's parameters): with P = rownorm(C o exp(scale Q K^T)), C the 0 / 1 /
 * (N/m) x multiplicity coefficients of the block mask, the samples and the causal recursion,
 *     dV = P^T dO,  dS = P o (dO V^T - rowsum(dO o O)),  dQ = scale dS K,  dK = scale dS^T Q.
 *   p->q, k, v       device, bf16 (fp32 inputs: HYPERATTN_UNSUPPORTED_SHAPE)
 *   p->out, p->lse   device, the forward call's results (read only here), out of p->out_dtype
 *   dout             device, bf16 [B, H, n, d]: gradient of the loss with respect to out
 *   dq, dk, dv       device, [B, H, n, d] of grad_dtype (HYPERATTN_BF16 or HYPERATTN_FP32), written;
 *                    16-byte aligned; must not alias any input
 * Gradients are accumulated in fp32 (in place for fp32 gradients, in the workspace otherwise) with
 * global reductions, so the low bits depend on the order in which tiles finish.  Enqueued on
 * p->stream like the forward pass; p->debug is ignored.  No gradient flows through lse. */
typedef struct hyperattn_grads {
  const void* dout;
  void* dq;
  void* dk;
  void* dv;
  int grad_dtype;
} hyperattn_grads;
int hyperattn_backward(const hyperattn_params* p, const hyperattn_grads* grads);
/* Bytes of device scratch hyperattn_backward needs (host-side, like hyperattn_workspace_bytes). */
int hyperattn_backward_workspace_bytes(const hyperattn_params* p, int grad_dtype, size_t* bytes);

/* Bytes of device scratch hyperattn_forward_ex needs for these shapes (host-side; only the
 * shape members, dtype and out_dtype of *p are read). */
int hyperattn_workspace_bytes(const hyperattn_params* p, size_t* bytes);

/* Host-side: writes the d x hash_bits direction matrix of Def. 1's hash (row-major,
 * entry [k*hash_bits + t] = coordinate k of direction t) that a call with this seed uses. */
int hyperattn_get_projections(int d, int hash_bits, uint64_t seed, float* host_out);
/* The same for the directions of recursion node `node`'s own (hyperattn_params.node_directions). */
int hyperattn_get_node_projections(int d, int hash_bits, uint64_t seed, int node, float* host_out);

/* Synchronises `stream` and reports the device status word (0, or
 * HYPERATTN_DEVICE_TIMEOUT if a kernel's bounded wait gave up since the last query) and
 * clears it.  While the word is set, attention tiles of later launches return without
 * computing, so a caller that saw a timeout must not use the outputs written since. */
int hyperattn_last_device_status(void* stream, int* status);

/* Stage timing.  While enabled, every forward call brackets each stage with CUDA events
 * on its stream and hyperattn_profile_read() (which synchronises those events) returns,
 * for every stage, the summed device milliseconds and launch count since the last
 * hyperattn_profile_reset().  Stage indices: */
enum {
  HYPERATTN_STAGE_CONVERT = 0, /* fp32 -> bf16 staging copy (fp32 inputs only) */
  HYPERATTN_STAGE_HASH = 1,    /* Def. 1 hash of Q and K rows + chunk histograms */
  HYPERATTN_STAGE_SAMPLE = 2,  /* Alg. 2 line 4: drawn inside the SORT_SCAN launch, so always 0 here */
  HYPERATTN_STAGE_SORT_SCAN = 3,
  HYPERATTN_STAGE_SORT_SCATTER = 4, /* Alg. 1 line 3 */
  HYPERATTN_STAGE_ATTENTION = 5,    /* block + sampled + causal-leaf contractions */
  HYPERATTN_STAGE_MERGE = 6,        /* Alg. 4 line 5 carried to outputs */
  HYPERATTN_STAGE_BACKWARD = 7,     /* hyperattn_backward: zeroing, <dO, O>, gradient tiles, conversion */
  HYPERATTN_NUM_STAGES = 8
};
typedef struct hyperattn_stage_times {
  float ms[HYPERATTN_NUM_STAGES];
  int launches[HYPERATTN_NUM_STAGES];
  int calls;
} hyperattn_stage_times;
/* on = 0: off; on = 1: every stage; any other value: only the stages s whose bit
 * (1 << (s + 1)) is set (fewer events on the stream between the kernels). */
int hyperattn_profile_enable(int on);
int hyperattn_profile_reset(void);
int hyperattn_profile_read(hyperattn_stage_times* out);

/* sortLSH of ONE bf16 matrix x[n, d] by an entry point that allocates nothing (the paper has no
 * counterpart to this entry point; what it computes is the hash and the argsort of
 * hyperattn_forward, for one matrix).  It is for callers that must not allocate device memory while
 * they run: a server that partitions HBM at start-up, a plug-in inside someone else's process, a loop
 * that may not take the driver's allocation locks.  Its scratch memory is a fixed array inside the
 * library image, 0.5 MB, which every GPU that loads the library holds until the process exits.
 *   x     device, [n, d] bf16 row-major, 16-byte aligned; d in {64, 128}; 1 <= hash_bits <= 8
 *   ids   device, uint8[n]  : bucket id of every row
 *   perm  device, int32[n]  : perm[p] = row at sorted position p (stable, ascending bucket id)
 *   rank  device, int32[n]  : inverse of perm
 * n may not exceed HYPERATTN_NOALLOC_MAX_ROWS; larger n returns HYPERATTN_UNSUPPORTED_SHAPE and
 * nothing is launched.  The caller owns x, ids, perm, rank.  Work is enqueued on `stream`; the
 * call does not synchronise and calls neither cudaMalloc / cudaFree nor any other allocating routine,
 * on the device or on the host.  The matrix is read once (it is hashed as the key side of a problem
 * without queries).  The first call on each device (with that device current) looks up the array's
 * device address and keeps it in a fixed table; make that first call outside any stream capture.
 * All calls share the one array: it keeps the previous call's contents (every word that is read is
 * rewritten first, so nothing needs clearing), and two calls whose kernels overlap on the GPU race
 * on it -- issue them on one stream or order them with events. */
#define HYPERATTN_NOALLOC_MAX_ROWS 262144
int hyperattn_sortlsh_noalloc(const void* x, int n, int d, int hash_bits, uint64_t seed,
                              uint8_t* ids, int32_t* perm, int32_t* rank, void* stream);

/* The quantity the paper's guarantee is stated in (Theorem 1; measured on real models in Sec. 4.3):
 *     alpha = n * max_j || D^-1 A e_j ||_2^2,
 * n times the largest squared column norm of the EXACT softmax matrix of every (batch, head), with the
 * causal mask M^C if causal != 0; the first skip_cols columns are left out of the maximum (Sec. 4.3 leaves
 * out the first 32 columns of causal language models, which hold heavy entries).  A diagnostic: it evaluates
 * the whole n x n_k matrix twice, so it is meant for a few thousand rows.
 *   q        device, bf16 [B, H, n, d];  k  device, bf16 [B, H, n_k, d] (n_k = 0 means n; causal needs n_k = n)
 *   alpha    device, float [B * H], written
 *   workspace device scratch of hyperattn_alpha_workspace_bytes(...) bytes, owned by the caller
 * softmax_scale <= 0 selects 1/sqrt(d).  Enqueued on `stream`; does not synchronise or allocate. */
int hyperattn_alpha(const void* q, const void* k, int B, int H, int n, int n_k, int d, float softmax_scale,
                    int causal, int skip_cols, float* alpha, void* workspace, size_t workspace_bytes, void* stream);
int hyperattn_alpha_workspace_bytes(int B, int H, int n, int n_k, size_t* bytes);

/* Frees the private workspaces and profiling events of every device. */
int hyperattn_release(void);

const char* hyperattn_status_string(int status);
int hyperattn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HYPERATTN_H_ */
