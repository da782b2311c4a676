// Combining the partial results of the causal recursion (Alg. 4 line 5 carried through to
// the outputs): a row of the second half of a recursion node adds the estimated row sums
// D~_21 + D~_C22, so its output is the sum of the partial outputs weighted by their share of
// the total row sum.  Every row owns one exact-leaf partial and one partial per recursion
// level at which it sits in a second half.  HBM-bound: reads the fp32 partials once, writes
// the final rows once.
#include <type_traits>

#include "common.cuh"

namespace hyperattn {
namespace {

struct MergeArgs {
  const void* part_o;        // rows of fp32, or of bf16 (PB)
  const float* part_lse;
  void* out; float* lse;
  Geometry g;
  int out_fp32;
};

// EPT consecutive entries of partial row k, starting at column EPT c (one 16-byte load, or 8 bytes for four bf16)
template <int D, bool PB, int EPT>
__device__ __forceinline__ void load_part(const void* base, size_t k, int c, float (&x)[EPT]) {
  if constexpr (PB && EPT == 8) {
    const uint4 w = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + k * D) + c);
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { x[2 * e] = __uint_as_float(u[e] << 16); x[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u); }
  } else if constexpr (PB) {
    const uint2 w = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(base) + k * D) + c);
    x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xffff0000u);
    x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xffff0000u);
  } else {
    const float4 w = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + k * D) + c);
    x[0] = w.x; x[1] = w.y; x[2] = w.z; x[3] = w.w;
  }
}

// LM: compile-time bound on the recursion depth (the loads of all levels are unrolled); PB: bf16 partials (then every
// thread owns eight columns, so that its loads stay 16 bytes wide; four for the deepest variant, to bound the registers)
template <int D, int LM, bool PB>
__global__ void __launch_bounds__(256) merge_kernel(MergeArgs a) {
  constexpr int EPT = (PB && LM <= 8) ? 8 : 4;
  constexpr int TPR = D / EPT;                     // threads per row
  const Geometry& g = a.g;
  // grid: x over the rows of a segment, y = segment
  const int seg = blockIdx.y;
  const int gt = blockIdx.x * blockDim.x + threadIdx.x;
  const int i = gt / TPR;
  const int c = gt % TPR;
  // (rows are never split between warps - TPR divides 32 - and a warp's rows past the end just idle: the shuffles
  // below name the row's own lanes only)
  const bool live = i < g.n;
  const unsigned rowmask = TPR >= 32 ? 0xffffffffu : (((1u << TPR) - 1u) << ((threadIdx.x & 31) / TPR * TPR));
  if (!live) return;
  const size_t row = (size_t)seg * g.n + i;
  // a node of level `level` has s = leaf << (L - 1 - level) rows, so the row's place in every level follows
  // from its leaf number by shifts
  const int leaf_no = i / g.leaf;
  const int in_leaf = i - leaf_no * g.leaf;
  // All loads of a row (its leaf partial and one partial per level at which it sits in a second
  // half) are issued before any is used: the kernel has nothing to hide their latency behind.
  float l[LM + 1];
  float x[LM + 1][EPT];
  // the row's log-sum-exp values are fetched by one lane each (lane t of the row takes partial t) and passed round
  float lmine = -INFINITY;
  if (c == 0) lmine = __ldcs(a.part_lse + row);
  load_part<D, PB, EPT>(a.part_o, row, c, x[0]);
#pragma unroll
  for (int level = 0; level < LM; ++level) {
    const int sh = g.L - 1 - level;                 // s = leaf << sh
    l[level + 1] = -INFINITY;
#pragma unroll
    for (int e = 0; e < EPT; ++e) x[level + 1][e] = 0.f;
    if (level < g.L && ((leaf_no >> sh) & 1)) {
      const int j = leaf_no >> (sh + 1);
      const int in_node = (leaf_no & ((1 << sh) - 1)) * g.leaf + in_leaf;      // i % s
      const size_t k = (size_t)g.G * g.n + ((size_t)level * g.G + seg) * g.nl + ((size_t)j << sh) * g.leaf + in_node;
      if (c == (level + 1) % TPR) lmine = (level + 1 < TPR) ? __ldcs(a.part_lse + k) : lmine;
      if (level + 1 >= TPR) l[level + 1] = __ldcs(a.part_lse + k);      // (more partials than lanes per row: fetched by every lane)
      load_part<D, PB, EPT>(a.part_o, k, c, x[level + 1]);
    }
  }
#pragma unroll
  for (int t = 0; t <= LM; ++t)
    if (t < TPR) l[t] = __shfl_sync(rowmask, lmine, (int)((threadIdx.x & 31) / TPR * TPR) + t);
  float mx = l[0];
#pragma unroll
  for (int t = 1; t <= LM; ++t) mx = fmaxf(mx, l[t]);
  float tot = 0.f;
#pragma unroll
  for (int t = 0; t <= LM; ++t) { l[t] = __expf(l[t] - mx); tot += l[t]; }   // exp(-inf) = 0 for the absent ones
  const float inv = 1.f / tot;
  float acc[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) acc[e] = 0.f;
#pragma unroll
  for (int t = 0; t <= LM; ++t) {
    const float w = l[t] * inv;
#pragma unroll
    for (int e = 0; e < EPT; ++e) acc[e] += w * x[t][e];
  }
  if (a.out_fp32) {
#pragma unroll
    for (int q4 = 0; q4 < EPT / 4; ++q4)
      __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + row * D + EPT * c) + q4,
             make_float4(acc[4 * q4], acc[4 * q4 + 1], acc[4 * q4 + 2], acc[4 * q4 + 3]));
  } else {
    uint32_t o[EPT / 2];
#pragma unroll
    for (int e = 0; e < EPT / 2; ++e) {
      __nv_bfloat162 t2 = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
      o[e] = *reinterpret_cast<uint32_t*>(&t2);
    }
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.out) + row * D + EPT * c;
    if constexpr (EPT == 8) __stcs(reinterpret_cast<uint4*>(dst), make_uint4(o[0], o[1], o[2], o[3]));
    else __stcs(reinterpret_cast<uint2*>(dst), make_uint2(o[0], o[1]));
  }
  if (c == 0) a.lse[row] = mx + __logf(tot);
}

}  // namespace

cudaError_t launch_merge(const Geometry& g, const Workspace& ws, void* out, float* lse, int out_fp32,
                         cudaStream_t st) {
  MergeArgs a; a.part_o = ws.part_o; a.part_lse = ws.part_lse; a.out = out; a.lse = lse; a.g = g; a.out_fp32 = out_fp32;
  const int ept = (ws.part_bf16 && g.L <= 8) ? 8 : 4;                   // columns per thread (see the kernel)
  const size_t threads = (size_t)g.n * (g.d / ept);
  const dim3 blocks((unsigned)((threads + 255) / 256), (unsigned)g.G);
  if (g.G > 65535) return cudaErrorInvalidValue;
  auto go = [&](auto kernel) { kernel<<<blocks, 256, 0, st>>>(a); };
  auto pick = [&](auto dtag, auto pbtag) {
    constexpr int D = decltype(dtag)::value;
    constexpr bool PB = decltype(pbtag)::value;
    if (g.L <= 3) go(merge_kernel<D, 3, PB>); else if (g.L <= 5) go(merge_kernel<D, 5, PB>); else if (g.L <= 8) go(merge_kernel<D, 8, PB>); else go(merge_kernel<D, kMaxLevelsMerge, PB>);
  };
  using std::integral_constant;
  if (g.d == 64) { if (ws.part_bf16) pick(integral_constant<int, 64>{}, integral_constant<bool, true>{}); else pick(integral_constant<int, 64>{}, integral_constant<bool, false>{}); }
  else { if (ws.part_bf16) pick(integral_constant<int, 128>{}, integral_constant<bool, true>{}); else pick(integral_constant<int, 128>{}, integral_constant<bool, false>{}); }
  return cudaGetLastError();
}

}  // namespace hyperattn
