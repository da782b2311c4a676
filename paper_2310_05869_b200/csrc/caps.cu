// Alg. 2 line 3: tau = max over the rows j of a random subset T of the sum of exp(scale <q_j, k>) over
// the keys k OUTSIDE row j's sorted block - the largest "unmasked" row sum among m probe rows.  One
// such maximum per (segment, recursion node); it feeds the upper cap C_i (line 6) and the lower cap
// tau / kappa (line 9) of the capped row-sum estimate.
//
// T is drawn as positions of the sorted query order (a uniform position is a uniform row; position p
// lies in group floor(p / b_q), so the row's block is known without an inverse permutation).  The
// kernel is a plain dense pass of m rows against all keys of the node on the warp-level tensor cores
// (mma.sync m16n8k16, fp32 accumulate): with N = 8 keys per product there is nothing for tcgen05 to
// win, and the pass costs m / (b + m) of the node's main work only because every probe row meets
// every key.  Results are kept as log2 of the row sum in the softmax's own scaled domain.
#include "attn_common.cuh"

namespace hyperattn {
namespace {

__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// (m, l) <- (m, l) (+) (m2, l2): log-sum-exp pairs in base 2
__device__ __forceinline__ void lse_merge(float& m, float& l, float m2, float l2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) return;
  l = l * ex2f(m - mn) + l2 * ex2f(m2 - mn);
  m = mn;
}
__device__ __forceinline__ void atomic_max_float(float* addr, float v) {
  if (v >= 0.f) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
  else atomicMin(reinterpret_cast<unsigned*>(addr), __float_as_uint(v));
}

struct TauArgs {
  const __nv_bfloat16 *q, *k;
  Geometry g;
  const int32_t *perm_q, *rank_k, *tpos;   // tpos: [G, nodes, m] positions in the sorted query order
  float* ltau;                             // [G, nodes] log2 of tau in the scaled domain; initialised to -inf
  float scale_log2;
};

// One CTA: 16 probe rows of one (segment, node) against all keys of the node; the 8 warps split the keys.
template <int D>
__global__ void __launch_bounds__(256) tau_kernel(const __grid_constant__ TauArgs a) {
  constexpr int KS = D / 16, CPL = D / 32;
  constexpr int U = D == 64 ? 4 : 2;               // 8-key blocks per step (independent loads in flight)
  __shared__ float s_m[8][16], s_l[8][16];
  const Geometry& g = a.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
  const int groups = (g.m + 15) / 16;
  int cta = blockIdx.x;
  const int rg = cta % groups; cta /= groups;
  const int node = cta % g.nodes;
  const int seg = cta / g.nodes;
  int level = 0, j = 0;
  if (g.causal) { level = 31 - __clz(node + 1); j = node + 1 - (1 << level); }
  int s, q0, k0;
  node_rows(g, level, j, s, q0, k0);
  const int nq = node_queries(g, s, q0);
  if (nq <= 0 || g.b >= s) return;                 // no such node, or a node that is one exact block
  const int bq = query_group(g.b, nq, s);
  const size_t slice = ((size_t)level * g.G + seg) * g.nl + (g.causal ? (size_t)j * s : 0);
  const int32_t* tp = a.tpos + ((size_t)seg * g.nodes + node) * g.m;

  // the two probe rows of this lane (rows gid and gid + 8 of the group) and the rank range of their blocks
  int row[2], lo[2], hi[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int idx = rg * 16 + gid + 8 * r;
    row[r] = -1; lo[r] = 0; hi[r] = 0;
    if (idx < g.m) {
      const int pos = tp[idx];
      row[r] = q0 + a.perm_q[slice + pos];
      lo[r] = (pos / bq) * g.b; hi[r] = lo[r] + g.b;
    }
  }
  // A fragments.  A dot product does not care in which order the coordinates are visited: k-slot
  // (2 tig + e) of step st holds coordinate 8 (tig + 4 (st >> 1)) + 4 (st & 1) + e (and slot 2 tig + 8 + e
  // the coordinate two further), for the probe rows and the keys alike, so every lane fetches 16-byte pieces.
  uint32_t af[KS][4];
  {
    const char* qb = reinterpret_cast<const char*>(a.q) + (size_t)seg * g.n * (D * 2);
    uint4 va[CPL], vb[CPL];
#pragma unroll
    for (int h = 0; h < CPL; ++h) {
      va[h] = row[0] >= 0 ? *reinterpret_cast<const uint4*>(qb + (size_t)row[0] * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
      vb[h] = row[1] >= 0 ? *reinterpret_cast<const uint4*>(qb + (size_t)row[1] * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int st = 0; st < KS; ++st) {
      af[st][0] = (st & 1) ? va[st >> 1].z : va[st >> 1].x;
      af[st][1] = (st & 1) ? vb[st >> 1].z : vb[st >> 1].x;
      af[st][2] = (st & 1) ? va[st >> 1].w : va[st >> 1].y;
      af[st][3] = (st & 1) ? vb[st >> 1].w : vb[st >> 1].y;
    }
  }
  const char* kb = reinterpret_cast<const char*>(a.k) + ((size_t)seg * g.nk + k0) * (D * 2);
  const int32_t* rk = a.rank_k + slice;
  float m2[2] = {-INFINITY, -INFINITY}, l2[2] = {0.f, 0.f};
  const int nblocks = (s + 7) / 8;
  for (int nb0 = warp * U; nb0 < nblocks; nb0 += 8 * U) {
    uint4 vk[U][CPL];
    int rnk[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int key = (nb0 + u) * 8 + gid;                     // the key whose coordinates this lane fetches
#pragma unroll
      for (int h = 0; h < CPL; ++h)
        vk[u][h] = key < s ? *reinterpret_cast<const uint4*>(kb + (size_t)key * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
      const int c = (nb0 + u) * 8 + 2 * tig;                    // the keys whose scores this lane receives
      rnk[u][0] = c < s ? rk[c] : -1;
      rnk[u][1] = c + 1 < s ? rk[c + 1] : -1;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int st = 0; st < KS; ++st)
        mma_16816(c, af[st], (st & 1) ? vk[u][st >> 1].z : vk[u][st >> 1].x, (st & 1) ? vk[u][st >> 1].w : vk[u][st >> 1].y);
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        float x[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int rank = rnk[u][e];
          const bool out = rank >= 0 && (rank < lo[r] || rank >= hi[r]);     // an existing key outside the row's block
          x[e] = out ? c[2 * r + e] * a.scale_log2 : -INFINITY;
        }
        const float mn = fmaxf(m2[r], fmaxf(x[0], x[1]));
        if (mn > -INFINITY) {
          l2[r] = l2[r] * ex2f(m2[r] - mn) + ex2f(x[0] - mn) + ex2f(x[1] - mn);
          m2[r] = mn;
        }
      }
    }
  }
  // the four lanes of a quad hold different keys of the same two rows; then the warps
#pragma unroll
  for (int r = 0; r < 2; ++r) {
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, m2[r], o), lo2 = __shfl_xor_sync(0xffffffffu, l2[r], o);
      lse_merge(m2[r], l2[r], mo, lo2);
    }
    if (tig == 0) { s_m[warp][gid + 8 * r] = m2[r]; s_l[warp][gid + 8 * r] = l2[r]; }
  }
  __syncthreads();
  if (warp == 0) {
    float best = -INFINITY;
    if (lane < 16 && rg * 16 + lane < g.m) {
      float m = s_m[0][lane], l = s_l[0][lane];
#pragma unroll
      for (int w = 1; w < 8; ++w) lse_merge(m, l, s_m[w][lane], s_l[w][lane]);
      if (m > -INFINITY && l > 0.f) best = m + log2f(l);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (lane == 0 && best > -INFINITY) atomic_max_float(a.ltau + (size_t)seg * g.nodes + node, best);
  }
}

}  // namespace

cudaError_t launch_tau(const AttnArgs& at, const int32_t* tpos, float* ltau, cudaStream_t st) {
  const Geometry& g = at.g;
  if (!g.sorted || g.m == 0 || g.nodes == 0) return cudaSuccess;
  TauArgs a;
  a.q = at.q; a.k = at.k; a.g = g; a.perm_q = at.perm_q; a.rank_k = at.rank_k; a.tpos = tpos; a.ltau = ltau;
  a.scale_log2 = at.scale_log2;
  const long long grid = (long long)g.G * g.nodes * ((g.m + 15) / 16);
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (g.d == 64) tau_kernel<64><<<(unsigned)grid, 256, 0, st>>>(a);
  else tau_kernel<128><<<(unsigned)grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hyperattn
