// Shared declarations of the HyperAttention forward library (sm_100a).
// Notation follows the paper: n rows, d head dimension, b block size, m sampled columns,
// r hash bits, G = B*H independent (batch, head) segments.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hyperattn {

constexpr int kSortChunk = 2048;      // rows per histogram / scatter chunk
constexpr int kBuckets = 256;         // 2^r with r <= 8
constexpr int kTileQ = 128;           // query rows per attention tile
constexpr int kMaxLevelsMerge = 24;   // deepest causal recursion supported

// ---- Philox4x32-10 (Salmon et al., SC'11); identical on host and device -------------
struct Philox4 { uint32_t x[4]; };

__host__ __device__ inline void mulhilo32(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
#ifdef __CUDA_ARCH__
  lo = a * b;
  hi = __umulhi(a, b);
#else
  uint64_t p = (uint64_t)a * b;
  lo = (uint32_t)p;
  hi = (uint32_t)(p >> 32);
#endif
}

__host__ __device__ inline Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int rnd = 0; rnd < 10; ++rnd) {
    if (rnd > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo32(0xD2511F53u, c0, hi0, lo0);
    mulhilo32(0xCD9E8D57u, c2, hi1, lo1);
    uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  Philox4 r; r.x[0] = c0; r.x[1] = c1; r.x[2] = c2; r.x[3] = c3;
  return r;
}
constexpr uint32_t kDomainDirections = 1, kDomainSamples = 2, kDomainRowSubset = 3;

// ---- geometry of one forward call, shared by all stages --------------------------------
// "unit" = the largest row range that never straddles a recursion node: a causal leaf of n0
// rows, or the whole segment.  Units are cut into chunks of at most kSortChunk rows; one
// hash CTA produces the ids and the 256-bin histogram of one chunk, one scatter CTA places it.
struct Geometry {
  int G, n, d;         // n: query rows per segment
  int nk;              // key / value rows per segment (n, unless a non-causal call has another number of keys)
  int npad;            // causal: leaf << L, the length whose halves the recursion cuts (>= n: rows beyond n do
                       // not exist, so the last leaf and the query side of a level's last node may be short);
                       // non-causal: n
  int b, m, r;
  int bq;              // rows per group of sorted queries of a full node: b, or ceil(b n / nk) for unequal sides
  int causal;          // 1: causal with L >= 1 levels or a single causal leaf
  int L;               // number of recursion levels with off-diagonal nodes (0: none)
  int leaf;            // rows per exact leaf (n if L == 0)
  int unit;            // rows per unit (query side; both sides of a causal call)
  int chunks_per_unit;
  int chunks_per_seg;  // (npad / unit) * chunks_per_unit
  int unit_k, chunks_per_unit_k, chunks_per_seg_k;   // the same for the key side
  int levels;          // sorted levels: L if causal, else 1 (0 if nothing is sorted)
  int nl;              // sorted rows per (level, segment, side): npad/2 causal, max(n, nk) non-causal
  int nodes;           // off-diagonal nodes per segment (heap-numbered)
  int sorted;          // 1 if any node needs sortLSH (some node has b < its size)
  int seg0;            // index, in the caller's tensor, of this call's first segment (the sampling counters carry it)
  int node_dirs;       // 1: every recursion node hashes with directions of its own: ids and chunk histograms exist
                       // once per level (a row is on one side of exactly one node per level)
};
// ids / histograms of a level start this many elements after those of level 0 (0: one set shared by all levels)
__host__ __device__ inline size_t ids_level_stride(const Geometry& g) { return g.node_dirs ? (size_t)g.G * ((size_t)g.n + g.nk) : 0; }
__host__ __device__ inline size_t hist_level_stride(const Geometry& g) { return g.node_dirs ? (size_t)g.G * (g.chunks_per_seg + g.chunks_per_seg_k) * kBuckets : 0; }

// sorted blocks of a node of s rows: ceil(s / b) of them, the last one with the remaining rows
// (Alg. 1 line 4: row i belongs to block floor(P(i) / b))
__host__ __device__ inline int node_blocks(int s, int b) { return (s + b - 1) / b; }
__host__ __device__ inline int block_len(int s, int b, int beta) { return (s - beta * b) < b ? (s - beta * b) : b; }

// node j of level l: number of keys s, first query row, first key row (non-causal: the whole segment)
__host__ __device__ inline void node_rows(const Geometry& g, int level, int j, int& s, int& q0, int& k0) {
  if (!g.causal) { s = g.nk; q0 = 0; k0 = 0; return; }
  s = g.npad >> (level + 1);
  q0 = (2 * j + 1) * s;
  k0 = 2 * j * s;
}
// query rows of a node whose nominal size is s and whose first query row is q0: s, unless the sequence
// ends inside it (the last node of a causal level) or the call has another number of queries than keys
__host__ __device__ inline int node_queries(const Geometry& g, int s, int q0) {
  if (!g.causal) return g.n;
  const int left = g.n - q0;
  return left < 0 ? 0 : (left < s ? left : s);
}
// rows per group of sorted queries when nq queries meet s keys in groups of b (Alg. 1 line 4 pairs group
// beta of either side; with nq != s the groups cover the same fraction of the sorted order): ceil(b nq / s)
__host__ __device__ inline int query_group(int b, int nq, int s) {
  return (int)(((long long)b * nq + s - 1) / s);
}
// per-side chunk geometry (side 0: queries, side 1: keys)
__host__ __device__ inline int side_rows(const Geometry& g, int side) { return side ? g.nk : g.n; }
__host__ __device__ inline int side_unit(const Geometry& g, int side) { return side ? g.unit_k : g.unit; }
__host__ __device__ inline int side_cpu(const Geometry& g, int side) { return side ? g.chunks_per_unit_k : g.chunks_per_unit; }
__host__ __device__ inline int side_cps(const Geometry& g, int side) { return side ? g.chunks_per_seg_k : g.chunks_per_seg; }
// chunks of one (level, segment) on a side: every node of the level (causal), or the whole side
__host__ __device__ inline int side_cpl(const Geometry& g, int side) { return g.causal ? (g.nl / g.unit) * g.chunks_per_unit : side_cps(g, side); }

// ---- stage launchers (each enqueues on `st`; returns cudaGetLastError()) ---------------
struct Workspace {
  __nv_bfloat16 *q16, *k16, *v16;  // bf16 staging of fp32 inputs (else null)
  __nv_bfloat16 *q16lo, *k16lo;    // second bf16 term of fp32 Q, K: x ~= x16 + x16lo
  uint8_t* ids;                    // queries [G, n], then keys [G, nk]
  uint32_t* hist;                  // queries [G, chunks_per_seg, 256], then keys [G, chunks_per_seg_k, 256]
  uint32_t* offs;                  // per side: [levels, G, chunks per (level,seg), 256]
  int32_t *perm_q, *perm_k, *rank_k;  // [levels, G, nl]
  int32_t* samples;                // [G, nodes, m]
  int32_t* tpos;                   // capped row sums: [G, nodes, m] probe positions (else null)
  float* ltau;                     // capped row sums: [G, nodes] log2 of the largest unmasked probe row sum
  void* part_o; float* part_lse;   // causal partials: leaf [G,n,(d)] then per level [G,nl,(d)]; rows of fp32 or bf16
  int part_bf16;
  int* status;                     // device status word
};

cudaError_t launch_convert(const float* src, __nv_bfloat16* hi, __nv_bfloat16* lo, size_t count, cudaStream_t st);
// w_host: the shared direction matrix; w_nodes (device, [nodes, d, r], g.node_dirs only): the nodes' own
cudaError_t launch_hash(const Geometry& g, const void* q, const void* k, int is_fp32, const float* w_host,
                        const Workspace& ws, unsigned long long* near_zero, cudaStream_t st, int side_mask = 3,
                        const float* w_nodes = nullptr);
// side_mask: bit 0 queries, bit 1 keys (3: both)
cudaError_t launch_sort_scan(const Geometry& g, const Workspace& ws, bool with_samples, uint64_t seed, cudaStream_t st, int side_mask = 3);
cudaError_t launch_sort_scatter(const Geometry& g, const Workspace& ws, cudaStream_t st, int side_mask = 3);
// side_mask for the hash as well (a side that is left out is neither read nor written)
cudaError_t launch_merge(const Geometry& g, const Workspace& ws, void* out, float* lse, int out_fp32,
                         cudaStream_t st);

}  // namespace hyperattn
