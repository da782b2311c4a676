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

template <int D>
__global__ void __launch_bounds__(256) merge_kernel(MergeArgs a) {
  constexpr int TPR = D / 4;                       // threads per row (one float4 each)
  const Geometry& g = a.g;
  const size_t rows = (size_t)g.G * g.n;
  const size_t gt = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t row = gt / TPR;
  const int c = (int)(gt % TPR);
  if (row >= rows) return;
  const int seg = (int)(row / g.n), i = (int)(row % g.n);
  size_t idx[kMaxLevelsMerge + 1];
  float l[kMaxLevelsMerge + 1];
  int cnt = 1;
  idx[0] = row;
  l[0] = a.part_lse[row];
  float mx = l[0];
  for (int level = 0; level < g.L; ++level) {
    const int s = g.n >> (level + 1);
    if ((i / s) & 1) {
      const int j = i / (2 * s);
      const size_t k = (size_t)g.G * g.n + ((size_t)level * g.G + seg) * g.nl + (size_t)j * s + (i % s);
      idx[cnt] = k;
      l[cnt] = a.part_lse[k];
      mx = fmaxf(mx, l[cnt]);
      ++cnt;
    }
  }
  float tot = 0.f;
  for (int t = 0; t < cnt; ++t) { l[t] = __expf(l[t] - mx); tot += l[t]; }
  const float inv = 1.f / tot;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int t = 0; t < cnt; ++t) {
    const float4 x = reinterpret_cast<const float4*>(a.part_o + idx[t] * D)[c];
    const float w = l[t] * inv;
    acc.x += w * x.x; acc.y += w * x.y; acc.z += w * x.z; acc.w += w * x.w;
  }
  if (a.out_fp32) {
    reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + row * D)[c] = acc;
  } else {
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.out) + row * D)[c] = o;
  }
  if (c == 0) a.lse[row] = mx + __logf(tot);
}

}  // namespace

cudaError_t launch_merge(const Geometry& g, const Workspace& ws, void* out, float* lse, int out_fp32,
                         cudaStream_t st) {
  MergeArgs a; a.part_o = ws.part_o; a.part_lse = ws.part_lse; a.out = out; a.lse = lse; a.g = g; a.out_fp32 = out_fp32;
  const size_t threads = (size_t)g.G * g.n * (g.d / 4);
  const unsigned blocks = (unsigned)((threads + 255) / 256);
  if (g.d == 64) merge_kernel<64><<<blocks, 256, 0, st>>>(a);
  else merge_kernel<128><<<blocks, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hyperattn
