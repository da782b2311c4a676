// Combining the partial results of the causal recursion (Alg. 4 line 5 carried through to
// the outputs): a row of the second half of a recursion node adds the estimated row sums
// D~_21 + D~_C22, so its output is the sum of the partial outputs weighted by their share of
// the total row sum.  Every row owns one exact-leaf partial and one partial per recursion
// level at which it sits in a second half.  HBM-bound: reads the fp32 partials once, writes
// the final rows once.
#include "common.cuh"

namespace hyperattn {
namespace {

struct MergeArgs {
  const float *part_o, *part_lse;
  void* out; float* lse;
  Geometry g;
  int out_fp32;
};

// LM: compile-time bound on the recursion depth (the loads of all levels are unrolled)
template <int D, int LM>
__global__ void __launch_bounds__(256) merge_kernel(MergeArgs a) {
  constexpr int TPR = D / 4;                       // threads per row (one float4 each)
  const Geometry& g = a.g;
  // grid: x over the rows of a segment, y = segment
  const int seg = blockIdx.y;
  const int gt = blockIdx.x * blockDim.x + threadIdx.x;
  const int i = gt / TPR;
  const int c = gt % TPR;
  if (i >= g.n) return;
  const size_t row = (size_t)seg * g.n + i;
  // n = leaf * 2^L: a node of level `level` has s = leaf << (L - 1 - level) rows, so the row's
  // place in every level follows from its leaf number by shifts
  const int leaf_no = i / g.leaf;
  const int in_leaf = i - leaf_no * g.leaf;
  // All loads of a row (its leaf partial and one partial per level at which it sits in a second
  // half) are issued before any is used: the kernel has nothing to hide their latency behind.
  float l[LM + 1];
  float4 x[LM + 1];
  l[0] = __ldcs(a.part_lse + row);
  x[0] = __ldcs(reinterpret_cast<const float4*>(a.part_o + row * D) + c);
#pragma unroll
  for (int level = 0; level < LM; ++level) {
    const int sh = g.L - 1 - level;                 // s = leaf << sh
    l[level + 1] = -INFINITY;
    x[level + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (level < g.L && ((leaf_no >> sh) & 1)) {
      const int j = leaf_no >> (sh + 1);
      const int in_node = (leaf_no & ((1 << sh) - 1)) * g.leaf + in_leaf;      // i % s
      const size_t k = (size_t)g.G * g.n + ((size_t)level * g.G + seg) * g.nl + ((size_t)j << sh) * g.leaf + in_node;
      l[level + 1] = __ldcs(a.part_lse + k);
      x[level + 1] = __ldcs(reinterpret_cast<const float4*>(a.part_o + k * D) + c);
    }
  }
  float mx = l[0];
#pragma unroll
  for (int t = 1; t <= LM; ++t) mx = fmaxf(mx, l[t]);
  float tot = 0.f;
#pragma unroll
  for (int t = 0; t <= LM; ++t) { l[t] = __expf(l[t] - mx); tot += l[t]; }   // exp(-inf) = 0 for the absent ones
  const float inv = 1.f / tot;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int t = 0; t <= LM; ++t) {
    const float w = l[t] * inv;
    acc.x += w * x[t].x; acc.y += w * x[t].y; acc.z += w * x[t].z; acc.w += w * x[t].w;
  }
  if (a.out_fp32) {
    __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + row * D) + c, acc);
  } else {
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
    __stcs(reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.out) + row * D) + c, o);
  }
  if (c == 0) a.lse[row] = mx + __logf(tot);
}

}  // namespace

cudaError_t launch_merge(const Geometry& g, const Workspace& ws, void* out, float* lse, int out_fp32,
                         cudaStream_t st) {
  MergeArgs a; a.part_o = ws.part_o; a.part_lse = ws.part_lse; a.out = out; a.lse = lse; a.g = g; a.out_fp32 = out_fp32;
  const size_t threads = (size_t)g.n * (g.d / 4);
  const dim3 blocks((unsigned)((threads + 255) / 256), (unsigned)g.G);
  if (g.G > 65535) return cudaErrorInvalidValue;
  auto go = [&](auto kernel) { kernel<<<blocks, 256, 0, st>>>(a); };
  if (g.d == 64) {
    if (g.L <= 3) go(merge_kernel<64, 3>); else if (g.L <= 5) go(merge_kernel<64, 5>); else if (g.L <= 8) go(merge_kernel<64, 8>); else go(merge_kernel<64, kMaxLevelsMerge>);
  } else {
    if (g.L <= 3) go(merge_kernel<128, 3>); else if (g.L <= 5) go(merge_kernel<128, 5>); else if (g.L <= 8) go(merge_kernel<128, 8>); else go(merge_kernel<128, kMaxLevelsMerge>);
  }
  return cudaGetLastError();
}

}  // namespace hyperattn
