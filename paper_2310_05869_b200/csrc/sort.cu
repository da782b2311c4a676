// sortLSH permutations (Alg. 1 line 3) and sampled columns (Alg. 2 line 4).
//
// The argsort is a stable counting sort: bucket ids have at most 256 values, so one pass of
//   per-chunk histogram (done by the hash kernel) -> per-node exclusive scan -> stable scatter
// orders every (level, segment, node, side) slice.  A chunk never straddles a recursion
// node, so the histogram of a chunk is the same at every level of the causal recursion and
// only the scan differs per level.  Ties keep the original row order, which makes the
// permutation unique.
#include "common.cuh"

namespace hyperattn {
namespace {

struct SortArgs {
  const uint8_t* ids;     // queries [G, n], then keys [G, nk]
  const uint32_t* hist;   // queries [G, chunks_per_seg, 256], then keys [G, chunks_per_seg_k, 256]
  uint32_t* offs;         // queries [levels, G, chunks per (level, segment), 256], then the same for keys
  int32_t *perm_q, *perm_k, *rank_k;  // [levels, G, nl]
  Geometry g;
  int side_mask;          // bit s set: side s is sorted (both, unless a caller wants one side only)
};

// chunk index (within a segment) of the first chunk of node j's query (side 0) or key (side 1) rows
// (chunks that lie beyond the last row have empty histograms and place nothing)
__device__ __forceinline__ int node_first_chunk(const Geometry& g, int level, int j, int side, int& nchunks) {
  if (!g.causal) { nchunks = side_cps(g, side); return 0; }
  int s, q0, k0;
  node_rows(g, level, j, s, q0, k0);
  nchunks = (s / g.unit) * g.chunks_per_unit;
  return ((side == 0 ? q0 : k0) / g.unit) * g.chunks_per_unit;
}
__device__ __forceinline__ size_t side_hist_base(const Geometry& g, int side) { return side ? (size_t)g.G * g.chunks_per_seg * kBuckets : 0; }
__device__ __forceinline__ size_t side_offs_base(const Geometry& g, int side) { return side ? (size_t)g.levels * g.G * side_cpl(g, 0) * kBuckets : 0; }
__device__ __forceinline__ size_t side_ids_base(const Geometry& g, int side) { return side ? (size_t)g.G * g.n : 0; }

struct SampleArgs {
  int32_t* samples;  // [G, nodes, m]
  int32_t* tpos;     // capped row sums only (else null): [G, nodes, m] probe positions of Alg. 2 line 2
  float* ltau;       // capped row sums only: [G, nodes], set to -inf here (the probe pass takes a maximum into it)
  Geometry g;
  uint32_t k0, k1;
};

// Alg. 2 line 4: m i.i.d. uniform key indices per (segment, node); word w of Philox call c is
// sample 4c + w, mapped to [0, N) by a 64-bit multiply-high.  `block` of `nblocks` blocks of 256 threads.
__device__ __forceinline__ void samples_body(const SampleArgs& a, int block, int nblocks) {
  const Geometry& g = a.g;
  const int calls = (g.m + 3) / 4;
  const size_t total = (size_t)g.G * g.nodes * calls;
  for (size_t i = (size_t)block * 256 + threadIdx.x; i < total; i += (size_t)nblocks * 256) {
    const int c = (int)(i % calls);
    const int nd = (int)((i / calls) % g.nodes);
    const int seg = (int)(i / ((size_t)calls * g.nodes));
    const int level = g.causal ? 31 - __clz(nd + 1) : 0;
    const uint32_t N = g.causal ? (uint32_t)(g.npad >> (level + 1)) : (uint32_t)g.nk;
    const Philox4 x = philox4x32_10((uint32_t)c, (uint32_t)(g.seg0 + seg), (uint32_t)nd, kDomainSamples, a.k0, a.k1);
    int32_t* dst = a.samples + ((size_t)seg * g.nodes + nd) * g.m;
#pragma unroll
    for (int w = 0; w < 4; ++w)
      if (4 * c + w < g.m) dst[4 * c + w] = (int32_t)__umulhi(x.x[w], N);
    if (a.tpos) {
      // Alg. 2 line 2: the probe rows T, m i.i.d. uniform positions of the node's sorted query order, from a
      // stream of their own (the node may have fewer queries than keys; none: nothing is read later)
      int s, q0, k0;
      node_rows(g, level, g.causal ? nd + 1 - (1 << level) : 0, s, q0, k0);
      const uint32_t NQ = (uint32_t)node_queries(g, s, q0);
      const Philox4 y = philox4x32_10((uint32_t)c, (uint32_t)(g.seg0 + seg), (uint32_t)nd, kDomainRowSubset, a.k0, a.k1);
      int32_t* dt = a.tpos + ((size_t)seg * g.nodes + nd) * g.m;
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (4 * c + w < g.m) dt[4 * c + w] = (int32_t)__umulhi(y.x[w], NQ);
      if (c == 0) a.ltau[(size_t)seg * g.nodes + nd] = -INFINITY;
    }
  }
}

// One CTA per (side, level, segment, node): thread v owns bucket v.  The launch carries the
// sampling as extra blocks (both are tiny and independent of each other).
__global__ void __launch_bounds__(256) sort_scan_kernel(SortArgs a, SampleArgs sa, int scan_blocks) {
  __shared__ uint32_t s_tot[kBuckets];
  if ((int)blockIdx.x >= scan_blocks) { samples_body(sa, blockIdx.x - scan_blocks, gridDim.x - scan_blocks); return; }
  const Geometry& g = a.g;
  const int v = threadIdx.x;
  int cta = blockIdx.x;
  // nodes of all levels are enumerated heap-style: per (side, seg): sum over levels of 2^level
  const int nodes_per = g.causal ? g.nodes : 1;
  const int nd = cta % nodes_per; cta /= nodes_per;
  const int seg = cta % g.G;
  const int side = cta / g.G;
  if (!((a.side_mask >> side) & 1)) return;
  int level = 0, j = nd;
  if (g.causal) { level = 31 - __clz(nd + 1); j = nd + 1 - (1 << level); }
  int nchunks;
  const int first = node_first_chunk(g, level, j, side, nchunks);
  const uint32_t* h = a.hist + level * hist_level_stride(g) + side_hist_base(g, side) + ((size_t)seg * side_cps(g, side) + first) * kBuckets;
  const int lvl_chunk0 = g.causal ? j * nchunks : 0;
  uint32_t* o = a.offs + side_offs_base(g, side) + (((size_t)level * g.G + seg) * side_cpl(g, side) + lvl_chunk0) * kBuckets;
  // pass 1: bucket totals of the node (eight loads in flight: the kernel is all latency)
  uint32_t tot = 0;
  for (int c0 = 0; c0 < nchunks; c0 += 8) {
    uint32_t t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = c0 + u < nchunks ? h[(size_t)(c0 + u) * kBuckets + v] : 0u;
#pragma unroll
    for (int u = 0; u < 8; ++u) tot += t[u];
  }
  // exclusive scan of the bucket totals over v
  s_tot[v] = tot;
  __syncthreads();
  for (int off = 1; off < kBuckets; off <<= 1) {
    const uint32_t add = v >= off ? s_tot[v - off] : 0u;
    __syncthreads();
    s_tot[v] += add;
    __syncthreads();
  }
  // pass 2: first position of bucket v in every chunk = buckets before v + the same bucket in earlier chunks
  uint32_t run = s_tot[v] - tot;
  for (int c0 = 0; c0 < nchunks; c0 += 8) {
    uint32_t t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = c0 + u < nchunks ? h[(size_t)(c0 + u) * kBuckets + v] : 0u;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (c0 + u < nchunks) o[(size_t)(c0 + u) * kBuckets + v] = run;
      run += t[u];
    }
  }
}

// One CTA per (side, level, segment, chunk of the level): stable placement of <= 2048 rows.
template <int R>
__global__ void __launch_bounds__(256) sort_scatter_kernel(SortArgs a) {
  __shared__ __align__(16) uint32_t s_cnt[8][kBuckets];   // per-warp running positions
  __shared__ uint8_t s_id[kSortChunk];
  const Geometry& g = a.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int cta = blockIdx.x;
  const int ctas0 = ((a.side_mask & 1) ? g.levels * g.G * side_cpl(g, 0) : 0);
  const int side = (cta >= ctas0 || !(a.side_mask & 1)) ? 1 : 0;
  if (side) cta -= ctas0;
  const int cpl = side_cpl(g, side);
  const int lc = cta % cpl; cta /= cpl;
  const int seg = cta % g.G;
  const int level = cta / g.G;
  // which node and which row range this chunk is
  int s, q0, k0, j = 0, nchunks_node = cpl;
  if (g.causal) {
    s = g.npad >> (level + 1);
    nchunks_node = (s / g.unit) * g.chunks_per_unit;
    j = lc / nchunks_node;
  }
  node_rows(g, level, j, s, q0, k0);
  const int cn = lc - j * nchunks_node;                  // chunk within the node
  const int cpu_s = side_cpu(g, side), unit_s = side_unit(g, side);
  const int u = cn / cpu_s, cu = cn % cpu_s;
  const int local0 = u * unit_s + cu * kSortChunk;       // first row, relative to the node
  const int row0 = (side == 0 ? q0 : k0) + local0;       // first row within the segment
  // (a chunk beyond the last row of the side has nothing to place)
  const int rows = min(min(kSortChunk, unit_s - cu * kSortChunk), side_rows(g, side) - row0);
  if (rows <= 0) return;

  const uint8_t* ids = a.ids + level * ids_level_stride(g) + side_ids_base(g, side) + (size_t)seg * side_rows(g, side) + row0;
  for (int i = tid; i < rows; i += 256) s_id[i] = ids[i];
  for (int i = tid; i < 8 * kBuckets / 4; i += 256) reinterpret_cast<uint4*>(&s_cnt[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  // per-warp histograms of consecutive sub-ranges of 256 rows
  const int wbeg = warp * (kSortChunk / 8);
  const int wend = min(rows, wbeg + kSortChunk / 8);
  for (int i = wbeg + lane; i < wend; i += 32) atomicAdd(&s_cnt[warp][s_id[i]], 1u);
  __syncthreads();
  {
    const uint32_t* o = a.offs + side_offs_base(g, side) + (((size_t)level * g.G + seg) * cpl + lc) * kBuckets;
    uint32_t run = o[tid];
#pragma unroll
    for (int w = 0; w < 8; ++w) { const uint32_t t = s_cnt[w][tid]; s_cnt[w][tid] = run; run += t; }
  }
  __syncthreads();
  const size_t slice = ((size_t)level * g.G + seg) * g.nl + (g.causal ? (size_t)j * s : 0);
  int32_t* perm = (side == 0 ? a.perm_q : a.perm_k) + slice;
  int32_t* rank = side == 1 ? a.rank_k + slice : nullptr;
  for (int i0 = wbeg; i0 < wend; i0 += 32) {
    const int i = i0 + lane;
    const bool act = i < wend;
    const uint32_t id = act ? s_id[i] : 0u;
    // lanes with the same bucket id: one ballot per id bit (ids have at most 8 bits; a generic
    // match.any costs several times more)
    uint32_t peers = __ballot_sync(0xffffffffu, act);
#pragma unroll
    for (int bit = 0; bit < R; ++bit) {                 // (ids have R bits)
      const uint32_t bal = __ballot_sync(0xffffffffu, (id >> bit) & 1u);
      peers &= ((id >> bit) & 1u) ? bal : ~bal;
    }
    const int before = __popc(peers & ((1u << lane) - 1u));
    uint32_t pos = 0;
    if (act) pos = s_cnt[warp][id] + before;
    __syncwarp();
    if (act && before == 0) s_cnt[warp][id] += __popc(peers);
    __syncwarp();
    if (act) {
      perm[pos] = local0 + i;
      if (rank) rank[local0 + i] = (int32_t)pos;
    }
  }
}

}  // namespace

static SortArgs make_sort_args(const Geometry& g, const Workspace& ws, int side_mask) {
  SortArgs a;
  a.ids = ws.ids; a.hist = ws.hist; a.offs = ws.offs;
  a.perm_q = ws.perm_q; a.perm_k = ws.perm_k; a.rank_k = ws.rank_k;
  a.g = g;
  a.side_mask = side_mask;
  return a;
}

// scan of the chunk histograms; with_samples: the same launch also draws the samples (Alg. 2 line 4)
cudaError_t launch_sort_scan(const Geometry& g, const Workspace& ws, bool with_samples, uint64_t seed, cudaStream_t st, int side_mask) {
  // (ws.tpos non-null: the launch also draws the probe rows of the capped row-sum estimate)
  if (!g.sorted) return cudaSuccess;
  const SortArgs a = make_sort_args(g, ws, side_mask);
  const int nodes_per = g.causal ? g.nodes : 1;
  const int scan_blocks = 2 * g.G * nodes_per;
  SampleArgs sa; sa.samples = ws.samples; sa.tpos = ws.tpos; sa.ltau = ws.ltau; sa.g = g; sa.k0 = (uint32_t)seed; sa.k1 = (uint32_t)(seed >> 32);
  int sample_blocks = 0;
  if (with_samples && g.nodes > 0 && g.m > 0) {
    const size_t total = (size_t)g.G * g.nodes * ((g.m + 3) / 4);
    const size_t blocks = (total + 255) / 256;
    sample_blocks = (int)(blocks < 1184 ? blocks : 1184);
  }
  sort_scan_kernel<<<scan_blocks + sample_blocks, 256, 0, st>>>(a, sa, scan_blocks);
  return cudaGetLastError();
}

cudaError_t launch_sort_scatter(const Geometry& g, const Workspace& ws, cudaStream_t st, int side_mask) {
  if (!g.sorted) return cudaSuccess;
  const SortArgs a = make_sort_args(g, ws, side_mask);
  const int grid = g.levels * g.G * (((side_mask & 1) ? side_cpl(g, 0) : 0) + ((side_mask & 2) ? side_cpl(g, 1) : 0));
  switch (g.r) {                                         // the hash width is a template parameter of the ballot loop
    case 1: sort_scatter_kernel<1><<<grid, 256, 0, st>>>(a); break;
    case 2: sort_scatter_kernel<2><<<grid, 256, 0, st>>>(a); break;
    case 3: sort_scatter_kernel<3><<<grid, 256, 0, st>>>(a); break;
    case 4: sort_scatter_kernel<4><<<grid, 256, 0, st>>>(a); break;
    case 5: sort_scatter_kernel<5><<<grid, 256, 0, st>>>(a); break;
    case 6: sort_scatter_kernel<6><<<grid, 256, 0, st>>>(a); break;
    case 7: sort_scatter_kernel<7><<<grid, 256, 0, st>>>(a); break;
    default: sort_scatter_kernel<8><<<grid, 256, 0, st>>>(a); break;
  }
  return cudaGetLastError();
}

}  // namespace hyperattn
