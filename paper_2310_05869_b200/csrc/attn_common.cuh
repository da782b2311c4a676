// Tile schedule shared by the attention kernels.
//
// One attention tile = 128 query rows against a list of key tiles.  Two kinds:
//   DENSE  contiguous query rows against a contiguous key range, optionally with the causal
//          mask M^C_ij = 1{i >= j}: the exact base case of the causal recursion (Alg. 4 read
//          with a base size), a problem that is a single block (b >= N), and nothing else.
//   NODE   128 consecutive *sorted* query positions of block beta of a HyperAttention problem:
//          keys are the b keys of sorted block beta (Alg. 1 line 4 / Sec. 4 block-diagonal
//          part) followed by the m sampled keys (Alg. 2 line 7), which carry the weight N/m
//          as an additive log2(N/m) on the logit, or minus infinity when the sampled key
//          lies in block beta itself (the factor 1 - M^H).
// All tiles of all recursion levels and all leaves of one forward call form one flat list
// so that a single launch covers them; heavy (leaf) tiles come first.
#pragma once
#include "common.cuh"

namespace hyperattn {

constexpr int kMaxLevels = 24;
constexpr int kMaxWeightedSamples = 512;   // sampled columns with weights of their own (sampling by value norms): table size
constexpr int kMaxNodeKeys = 2048;   // 2 * (b rounded up to 128) + (m rounded up to 128) must fit the key table

struct AttnArgs {
  const __nv_bfloat16 *q, *k, *v;    // [G, n, D]
  const __nv_bfloat16 *q_lo, *k_lo;  // second bf16 term of fp32 inputs (else null)
  Geometry g;
  float scale_log2;                  // softmax scale * log2(e)
  const int32_t *perm_q, *perm_k, *rank_k, *samples;
  void* part_o; float* part_lse;     // partial results, used when !direct: rows of fp32, or of bf16 when part_bf16
  int part_bf16;                     // (partials are kept in the type of the final output; their log-sum-exp always in fp32)
  void* out; float* lse;             // final results, used when direct
  int out_fp32;
  int direct;
  int precise;                       // softmax weights enter the P V product as bf16 hi + lo
  // Alg. 2 with its caps (lines 3, 6, 7, 9): capped != 0 switches them on for the sorted nodes
  int capped;
  float cap_scale;                   // the constant of line 6: C_i = cap_scale m / (N ln N) (masked_i + tau / kappa)
  float log2_kappa;
  const float* ltau;                 // [G, nodes] log2 tau in the scaled domain
  // sampled columns drawn with probabilities of their own (Lemma 2): log2 of the weight 1 / (m p) of every draw,
  // [G, nodes, m]; null: uniform sampling, weight N / m
  const float* sample_wlog;
  // dense (leaf) tiles
  int dense_causal;
  int tiles_per_leaf, leaves_per_seg, n_leaf_tiles;
  // node tiles, per level
  int level_start[kMaxLevels + 1];   // first tile index of each level (after the leaf tiles)
  int level_sorted[kMaxLevels];      // 1: sortLSH node tiles; 0: single-block node (dense tiles)
  int tiles_per_block;               // ceil(bq / 128): query tiles per group of sorted queries of a full node
  int total_tiles;
  // the same schedule in pairs of neighbouring query tiles (tcgen05 path)
  int pairs_per_leaf, n_leaf_pairs;
  int level_pair_start[kMaxLevels + 1];
  int level_paired[kMaxLevels];      // 1: CTAs of this level own two query tiles, 0: one
  int total_pairs;
  int* sched;                        // work counter of the launch (global memory, zero at launch): next item to hand out
};

struct TileDesc {
  int mode;            // 0 dense, 1 node
  int seg;
  int nq;              // valid query rows
  int q0;              // dense: first query row (segment-relative)
  int k0, nk;          // dense: key range; node: first key row of the node, N
  int causal;          // dense: apply j_local <= i_local
  int qk_off;          // dense causal: local index of the tile's first query row relative to k0
  int qnode0;          // node: first query row of the node (segment-relative)
  size_t slice;        // node: offset of this node's slice in perm_q / perm_k / rank_k
  int spos0;           // node: first sorted position of the tile
  int beta;            // node: block index
  int bq;              // node: rows per group of sorted queries (b, unless the node has fewer / more queries than keys)
  int node;            // node: heap index
  size_t orow_base;    // output row index = orow_base + (segment-relative query row + odelta)
  int odelta;
  int partial;         // 1: write part_o/part_lse, 0: write out/lse
};

__device__ __forceinline__ TileDesc decode_tile(const AttnArgs& a, int tile) {
  const Geometry& g = a.g;
  TileDesc t;
  t.partial = !a.direct;
  if (tile < a.n_leaf_tiles) {
    // leaf after leaf, the tiles of a leaf from the heaviest (last rows, most keys) to the lightest: the CTAs that run
    // at the same time work on a handful of neighbouring leaves, whose K / V rows - and, in the backward pass, whose
    // dK / dV accumulator rows, which every query tile of the leaf adds to - then stay in L2
    const int tt = a.tiles_per_leaf - 1 - tile % a.tiles_per_leaf;
    const int rem = tile / a.tiles_per_leaf;
    t.seg = rem / a.leaves_per_seg;
    const int leaf = rem % a.leaves_per_seg;
    t.mode = 0;
    // a leaf: the rows [k0, k0 + leaf) that exist; a non-causal call that is one block: all n queries against all nk keys
    t.k0 = leaf * g.leaf; t.nk = g.causal ? max(0, min(g.leaf, g.n - t.k0)) : g.nk;
    t.q0 = t.k0 + tt * kTileQ;
    t.nq = max(0, min(kTileQ, (g.causal ? t.nk : g.n) - tt * kTileQ));
    t.causal = a.dense_causal;
    t.qk_off = tt * kTileQ;
    t.orow_base = (size_t)t.seg * g.n; t.odelta = 0;
    return t;
  }
  int level = 0;
  while (level + 1 < g.levels && tile >= a.level_start[level + 1]) ++level;
  int idx = tile - a.level_start[level];
  int s, q0n, k0n;
  node_rows(g, level, 0, s, q0n, k0n);
  const int nodes_lvl = g.causal ? (1 << level) : 1;
  const size_t region = a.direct ? 0 : (size_t)g.G * g.n + (size_t)level * g.G * g.nl;
  if (a.level_sorted[level]) {
    const int tiles_node = node_blocks(s, g.b) * a.tiles_per_block;
    const int tn = idx % tiles_node; idx /= tiles_node;
    const int j = idx % nodes_lvl;
    t.seg = idx / nodes_lvl;
    node_rows(g, level, j, s, q0n, k0n);
    t.mode = 1;
    const int nqn = node_queries(g, s, q0n);
    t.bq = query_group(g.b, nqn, s);
    t.beta = tn / a.tiles_per_block;
    const int sub = tn % a.tiles_per_block;
    t.spos0 = t.beta * t.bq + sub * kTileQ;
    t.nq = t.bq > 0 ? max(0, min(kTileQ, block_len(nqn, t.bq, t.beta) - sub * kTileQ)) : 0;   // 0: the group has no such tile
    t.k0 = k0n; t.nk = s; t.qnode0 = q0n;
    t.slice = ((size_t)level * g.G + t.seg) * g.nl + (g.causal ? (size_t)j * s : 0);
    t.node = g.causal ? (1 << level) - 1 + j : 0;
    t.causal = 0; t.q0 = 0; t.qk_off = 0;
    if (a.direct) { t.orow_base = (size_t)t.seg * g.n; t.odelta = 0; }
    else { t.orow_base = region + (size_t)t.seg * g.nl + (size_t)j * s; t.odelta = -q0n; }
  } else {
    const int tiles_node = ((g.causal ? s : g.n) + kTileQ - 1) / kTileQ;
    const int tn = idx % tiles_node; idx /= tiles_node;
    const int j = idx % nodes_lvl;
    t.seg = idx / nodes_lvl;
    node_rows(g, level, j, s, q0n, k0n);
    t.mode = 0;
    t.k0 = k0n; t.nk = s;
    t.q0 = q0n + tn * kTileQ;
    t.nq = max(0, min(kTileQ, node_queries(g, s, q0n) - tn * kTileQ));
    t.causal = 0; t.qk_off = 0;
    if (a.direct) { t.orow_base = (size_t)t.seg * g.n; t.odelta = 0; }
    else { t.orow_base = region + (size_t)t.seg * g.nl + (size_t)j * s; t.odelta = -q0n; }
  }
  return t;
}

}  // namespace hyperattn
