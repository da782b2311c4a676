// Stage 1 of sortLSH (Def. 1; Alg. 1 line 2): bucket id of every query and key row.
//
//   p_t = <x, w_t>,  bit_t = [p_t > 0],  g = sum_t bit_t 2^t,  id = Gray rank of g.
//
// The kernel streams Q and K once (HBM-bound: d*e bytes in, 1 byte out per row) and also
// leaves a 256-bin histogram per chunk of rows, which is the first pass of the counting
// argsort (Alg. 1 line 3).
//
// bf16 rows: the projection [16 rows x d] . [d x 8] runs on the tensor cores
// (mma.sync m16n8k16, fp32 accumulate).  Each lane fetches its operands with 128-bit loads;
// because a dot product does not care in which order the coordinates are visited, the
// coordinates a lane happens to hold are assigned to MMA k-slots by a fixed permutation and
// the direction matrix is laid out with the same permutation.  The fp32 directions are split
// into three bf16 terms (w = w1 + w2 + w3 exactly), so the products are exact and only the
// fp32 accumulation rounds; signs can differ from an exact evaluation only where |p_t| is
// within ~1e-5 of zero.
#include "common.cuh"

namespace hyperattn {
namespace {

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Gray rank: h with h ^ (h >> 1) == g (prefix xor), 8-bit patterns.
__device__ __forceinline__ uint32_t gray_rank8(uint32_t g) {
  g ^= g >> 1; g ^= g >> 2; g ^= g >> 4;
  return g & 0xFFu;
}

struct HashArgs {
  const void* x[2];       // Q, K  [G, n, d]
  float w[128 * 8];       // [d, r] directions, passed by value (<= 4 KB of kernel parameters)
  uint8_t* ids;           // queries [G, n], then keys [G, nk]
  uint32_t* hist;         // queries [G, chunks_per_seg, 256], then keys [G, chunks_per_seg_k, 256]
  unsigned long long* near_zero;
  int G, r;
  int side_mask;          // bit s set: side s is hashed
  int n[2];               // rows per segment of either side
  int unit[2], chunks_per_unit[2], chunks_per_seg[2];
  // directions of every recursion node's own (causal calls): the grid covers every level; a chunk belongs to
  // node j = unit / (2 u) of its level (u units per half) and is hashed there if it lies on the side's half
  const float* w_nodes;   // [nodes, d, r] or null
  int levels, L, d;
  size_t ids_level_stride, hist_level_stride;
};

// which chunk a CTA owns: side, segment, first row, number of rows (0: the chunk lies beyond the last row)
struct ChunkPos { int side, seg, chunk, row0, rows, level, node; };
__device__ __forceinline__ ChunkPos chunk_of_cta(const HashArgs& a, int cta) {
  ChunkPos c;
  const int per_level = a.G * (a.chunks_per_seg[0] + a.chunks_per_seg[1]);
  c.level = cta / per_level; cta -= c.level * per_level;
  c.node = 0;
  const int ctas0 = a.G * a.chunks_per_seg[0];
  c.side = cta >= ctas0;
  if (c.side) cta -= ctas0;
  c.chunk = cta % a.chunks_per_seg[c.side];
  c.seg = cta / a.chunks_per_seg[c.side];
  const int unit_idx = c.chunk / a.chunks_per_unit[c.side], cu = c.chunk % a.chunks_per_unit[c.side];
  c.row0 = unit_idx * a.unit[c.side] + cu * kSortChunk;
  c.rows = max(0, min(min(kSortChunk, a.unit[c.side] - cu * kSortChunk), a.n[c.side] - c.row0));
  if (a.w_nodes) {
    // level l: nodes of 2 u units, u = 2^(L - 1 - l); queries live in the second half, keys in the first
    const int u = 1 << (a.L - 1 - c.level);
    const int j = unit_idx / (2 * u);
    const bool second = (unit_idx / u) & 1;
    c.node = (1 << c.level) - 1 + j;
    if (second != (c.side == 0)) c.rows = -1;          // this side of the level does not hold the chunk: nothing to do
  }
  return c;
}
__device__ __forceinline__ size_t ids_base(const HashArgs& a, const ChunkPos& c) {
  return c.level * a.ids_level_stride + (c.side ? (size_t)a.G * a.n[0] : 0) + (size_t)c.seg * a.n[c.side] + c.row0;
}
__device__ __forceinline__ size_t hist_base(const HashArgs& a, const ChunkPos& c) {
  return c.level * a.hist_level_stride + ((c.side ? (size_t)a.G * a.chunks_per_seg[0] : 0) + (size_t)c.seg * a.chunks_per_seg[c.side] + c.chunk) * kBuckets;
}

// One CTA = one chunk (<= kSortChunk rows of one side of one segment).  Each warp walks over
// groups of 16 rows; the loads of the next group are issued before the MMAs of the current
// one, and the direction fragments live in shared memory (one 8-byte read per MMA) instead
// of 48 registers, so that two to four CTAs fit an SM and ~128 KB of loads are in flight.
template <int D>
__global__ void __launch_bounds__(256, D == 64 ? 4 : 3) hash_bf16_kernel(const __grid_constant__ HashArgs a) {
  constexpr int KS = D / 16;             // MMA k-steps
  constexpr int CPL = D / 32;            // 16-byte chunks per lane per row
  __shared__ __align__(16) uint8_t s_ids[kSortChunk];
  __shared__ uint32_t s_hist[kBuckets];
  __shared__ uint2 s_bw[3][KS][32];      // [split][k-step][lane] -> (b0, b1) of that lane

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const ChunkPos cp = chunk_of_cta(a, blockIdx.x);
  const int side = cp.side, seg = cp.seg, row0 = cp.row0, rows = cp.rows;
  if (!((a.side_mask >> side) & 1) || rows < 0) return;
  const float* wsrc = a.w_nodes ? a.w_nodes + (size_t)cp.node * (D * a.r) : a.w;

  s_hist[tid] = 0;

  const char* base = reinterpret_cast<const char*>(a.x[side]) + ((size_t)seg * a.n[side] + row0) * (D * 2);
  unsigned nz = 0;
  const int groups = (rows + 15) >> 4;
  uint4 xa[CPL], xb[CPL];
  auto load_group = [&](int grp, uint4 (&pa)[CPL], uint4 (&pb)[CPL]) {
    const int ra = grp * 16 + gid, rb = ra + 8;
#pragma unroll
    for (int h = 0; h < CPL; ++h) {
      pa[h] = (grp < groups && ra < rows) ? ldg_stream(base + (size_t)ra * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
      pb[h] = (grp < groups && rb < rows) ? ldg_stream(base + (size_t)rb * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
    }
  };
  load_group(warp, xa, xb);                           // the first rows are on their way while the fragments are built

  // Direction fragments.  k-slot (step s, half h, element e) of lane (gid, tig) holds
  // coordinate 8*(tig + 4*(s>>1)) + 2*(2*(s&1) + h) + e; column gid is direction gid.
  for (int idx = tid; idx < KS * 32; idx += 256) {
    const int s = idx >> 5, l = idx & 31;
    const int lg = l >> 2, lt = l & 3;
    uint32_t packed[3][2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float t1[2], t2[2], t3[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int coord = 8 * (lt + 4 * (s >> 1)) + 2 * (2 * (s & 1) + h) + e;
        const float w = (lg < a.r) ? wsrc[coord * a.r + lg] : 0.f;
        t1[e] = __bfloat162float(__float2bfloat16_rn(w));
        const float r1 = w - t1[e];
        t2[e] = __bfloat162float(__float2bfloat16_rn(r1));
        t3[e] = __bfloat162float(__float2bfloat16_rn(r1 - t2[e]));
      }
      packed[0][h] = pack_bf16(t1[0], t1[1]);
      packed[1][h] = pack_bf16(t2[0], t2[1]);
      packed[2][h] = pack_bf16(t3[0], t3[1]);
    }
#pragma unroll
    for (int sp = 0; sp < 3; ++sp) s_bw[sp][s][l] = make_uint2(packed[sp][0], packed[sp][1]);
  }
  __syncthreads();

  for (int grp = warp; grp < groups; grp += 8) {
    const int ra = grp * 16 + gid, rb = ra + 8;
    uint4 na[CPL], nb[CPL];
    load_group(grp + 8, na, nb);                      // in flight while this group is multiplied
    float hi[4] = {0.f, 0.f, 0.f, 0.f}, lo[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint4 va = xa[s >> 1], vb = xb[s >> 1];
      uint32_t af[4];
      af[0] = (s & 1) ? va.z : va.x;   // row gid,   half 0
      af[1] = (s & 1) ? vb.z : vb.x;   // row gid+8, half 0
      af[2] = (s & 1) ? va.w : va.y;   // row gid,   half 1
      af[3] = (s & 1) ? vb.w : vb.y;   // row gid+8, half 1
      const uint2 w3 = s_bw[2][s][lane], w2 = s_bw[1][s][lane], w1 = s_bw[0][s][lane];
      mma_bf16_16816(lo, af, w3.x, w3.y);
      mma_bf16_16816(lo, af, w2.x, w2.y);
      mma_bf16_16816(hi, af, w1.x, w1.y);
    }
    // lane holds p[row gid][2tig], p[gid][2tig+1], p[gid+8][2tig], p[gid+8][2tig+1]
    float p[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = hi[i] + lo[i];
    uint32_t ga = (p[0] > 0.f ? 1u : 0u) << (2 * tig) | (p[1] > 0.f ? 1u : 0u) << (2 * tig + 1);
    uint32_t gb = (p[2] > 0.f ? 1u : 0u) << (2 * tig) | (p[3] > 0.f ? 1u : 0u) << (2 * tig + 1);
    if (a.near_zero) {
      if (2 * tig < a.r) { nz += (ra < rows && fabsf(p[0]) < 1e-4f); nz += (rb < rows && fabsf(p[2]) < 1e-4f); }
      if (2 * tig + 1 < a.r) { nz += (ra < rows && fabsf(p[1]) < 1e-4f); nz += (rb < rows && fabsf(p[3]) < 1e-4f); }
    }
    ga |= __shfl_xor_sync(0xffffffffu, ga, 1); ga |= __shfl_xor_sync(0xffffffffu, ga, 2);
    gb |= __shfl_xor_sync(0xffffffffu, gb, 1); gb |= __shfl_xor_sync(0xffffffffu, gb, 2);
    if (tig == 0 && ra < rows) { const uint32_t id = gray_rank8(ga); s_ids[ra] = (uint8_t)id; atomicAdd(&s_hist[id], 1u); }
    if (tig == 1 && rb < rows) { const uint32_t id = gray_rank8(gb); s_ids[rb] = (uint8_t)id; atomicAdd(&s_hist[id], 1u); }
#pragma unroll
    for (int h = 0; h < CPL; ++h) { xa[h] = na[h]; xb[h] = nb[h]; }
  }
  if (a.near_zero) {
#pragma unroll
    for (int o = 16; o; o >>= 1) nz += __shfl_xor_sync(0xffffffffu, nz, o);
    if (lane == 0 && nz) atomicAdd(a.near_zero, (unsigned long long)nz);
  }
  __syncthreads();
  uint8_t* dst = a.ids + ids_base(a, cp);
  if ((rows & 15) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
    for (int i = tid; i < rows / 16; i += 256)
      reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(s_ids)[i];
  } else {
    for (int i = tid; i < rows; i += 256) dst[i] = s_ids[i];
  }
  a.hist[hist_base(a, cp) + tid] = s_hist[tid];
}

// fp32 rows (small problems): one thread per row, plain fp32 FMA in coordinate order.
__global__ void __launch_bounds__(256) hash_fp32_kernel(const __grid_constant__ HashArgs a, int d) {
  __shared__ float s_w[128 * 8];
  __shared__ uint32_t s_hist[kBuckets];
  const int tid = threadIdx.x;
  const ChunkPos cp = chunk_of_cta(a, blockIdx.x);
  const int side = cp.side, seg = cp.seg, row0 = cp.row0, rows = cp.rows;
  if (!((a.side_mask >> side) & 1) || rows < 0) return;
  const float* wsrc = a.w_nodes ? a.w_nodes + (size_t)cp.node * (d * a.r) : a.w;
  s_hist[tid] = 0;
  for (int i = tid; i < d * a.r; i += 256) s_w[i] = wsrc[i];
  __syncthreads();
  const float* base = reinterpret_cast<const float*>(a.x[side]) + ((size_t)seg * a.n[side] + row0) * d;
  uint8_t* dst = a.ids + ids_base(a, cp);
  unsigned long long nz = 0;
  for (int row = tid; row < rows; row += 256) {
    float p[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const float4* xr = reinterpret_cast<const float4*>(base + (size_t)row * d);
    for (int c = 0; c < d / 4; ++c) {
      const float4 x = xr[c];
      const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int t = 0; t < 8; ++t)
          if (t < a.r) p[t] = fmaf(xs[e], s_w[(4 * c + e) * a.r + t], p[t]);
    }
    uint32_t g = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t)
      if (t < a.r) { g |= (p[t] > 0.f ? 1u : 0u) << t; nz += fabsf(p[t]) < 1e-4f; }
    const uint32_t id = gray_rank8(g);
    dst[row] = (uint8_t)id;
    atomicAdd(&s_hist[id], 1u);
  }
  if (a.near_zero && nz) atomicAdd(a.near_zero, nz);
  __syncthreads();
  a.hist[hist_base(a, cp) + tid] = s_hist[tid];
}

// fp32 -> bf16 staging; `lo` (optional) receives the rounding remainder as a second bf16 term
__global__ void convert_kernel(const float4* __restrict__ src, uint2* __restrict__ hi, uint2* __restrict__ lo,
                               size_t count4) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 x = src[i];
    const float xs[4] = {x.x, x.y, x.z, x.w};
    float h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { h[e] = __bfloat162float(__float2bfloat16_rn(xs[e])); l[e] = xs[e] - h[e]; }
    hi[i] = make_uint2(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]));
    if (lo) lo[i] = make_uint2(pack_bf16(l[0], l[1]), pack_bf16(l[2], l[3]));
  }
}

}  // namespace

cudaError_t launch_convert(const float* src, __nv_bfloat16* hi, __nv_bfloat16* lo, size_t count, cudaStream_t st) {
  const size_t count4 = count / 4;
  const size_t want = (count4 + 255) / 256;
  const int blocks = (int)(want < 148 * 16 ? (want ? want : 1) : 148 * 16);
  convert_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(hi),
                                         reinterpret_cast<uint2*>(lo), count4);
  return cudaGetLastError();
}

cudaError_t launch_hash(const Geometry& g, const void* q, const void* k, int is_fp32, const float* w_host,
                        const Workspace& ws, unsigned long long* near_zero, cudaStream_t st, int side_mask, const float* w_nodes) {
  HashArgs a;
  a.side_mask = side_mask;
  a.w_nodes = g.node_dirs ? w_nodes : nullptr;
  a.levels = g.node_dirs ? g.levels : 1; a.L = g.L; a.d = g.d;
  a.ids_level_stride = ids_level_stride(g); a.hist_level_stride = hist_level_stride(g);
  for (int i = 0; i < g.d * g.r; ++i) a.w[i] = w_host[i];
  a.x[0] = q; a.x[1] = k; a.ids = ws.ids; a.hist = ws.hist; a.near_zero = near_zero;
  a.G = g.G; a.r = g.r;
  for (int s = 0; s < 2; ++s) {
    a.n[s] = side_rows(g, s); a.unit[s] = side_unit(g, s);
    a.chunks_per_unit[s] = side_cpu(g, s); a.chunks_per_seg[s] = side_cps(g, s);
  }
  const int grid = a.levels * g.G * (g.chunks_per_seg + g.chunks_per_seg_k);
  if (is_fp32) hash_fp32_kernel<<<grid, 256, 0, st>>>(a, g.d);
  else if (g.d == 64) hash_bf16_kernel<64><<<grid, 256, 0, st>>>(a);
  else hash_bf16_kernel<128><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hyperattn
