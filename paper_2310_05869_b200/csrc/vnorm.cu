// Sampling the residual's columns by squared row norms of V (Lemma 2) instead of uniformly (Sec. 4):
//   p_l = ||V_l||^2 / ||V||_F^2 over the keys of a (segment, recursion node), m i.i.d. draws, weight
//   1 / (m p_l) per draw (the rows of Lemma 2's sampling matrix S, squared).
// Indices must be reproducible bit for bit, so the distribution is made of integers: the squared norm
// of a row is accumulated in fp32 in coordinate order (bf16 squares are exact in fp32) and cut to a
// multiple of 2^-12; cumulative sums are 64-bit integers; a draw is the first key whose cumulative
// weight exceeds floor(x * total / 2^32), x the Philox word the uniform sampler would have used.
// Three small kernels: weights (streams V once), per-segment cumulative sums, draws.
#include "common.cuh"

namespace hyperattn {
namespace {

constexpr float kNormScale = 4096.f;      // 2^12

// one thread per key row
template <int D>
__global__ void __launch_bounds__(256) vnorm_weights_kernel(const __nv_bfloat16* __restrict__ v, uint32_t* __restrict__ wq, size_t rows) {
  const size_t row = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (row >= rows) return;
  const uint4* src = reinterpret_cast<const uint4*>(v + row * D);
  float acc = 0.f;
#pragma unroll
  for (int c = 0; c < D / 8; ++c) {
    const uint4 x = src[c];
    const uint32_t words[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float lo = __uint_as_float(words[e] << 16), hi = __uint_as_float(words[e] & 0xffff0000u);
      acc = __fadd_rn(acc, __fmul_rn(lo, lo));          // (coordinate order, no fused multiply-add: the stated arithmetic)
      acc = __fadd_rn(acc, __fmul_rn(hi, hi));
    }
  }
  wq[row] = (uint32_t)(acc * kNormScale);               // exact scaling, truncation = floor (acc >= 0)
}

// One CTA per segment: cum[seg][0] = 0, cum[seg][i + 1] = wq[seg][0] + ... + wq[seg][i] (64-bit).
__global__ void __launch_bounds__(1024) vnorm_scan_kernel(const uint32_t* __restrict__ wq, unsigned long long* __restrict__ cum, int nk) {
  __shared__ unsigned long long s_warp[32];
  __shared__ unsigned long long s_base;
  const int seg = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* w = wq + (size_t)seg * nk;
  unsigned long long* c = cum + (size_t)seg * (nk + 1);
  if (tid == 0) { s_base = 0; c[0] = 0; }
  __syncthreads();
  for (int i0 = 0; i0 < nk; i0 += 4096) {
    const int i = i0 + 4 * tid;
    unsigned long long x[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) x[e] = i + e < nk ? w[i + e] : 0ull;
    x[1] += x[0]; x[2] += x[1]; x[3] += x[2];
    unsigned long long run = x[3];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, run, o);
      if (lane >= o) run += t;
    }
    if (lane == 31) s_warp[warp] = run;
    __syncthreads();
    if (warp == 0) {
      unsigned long long t = s_warp[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long u = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += u;
      }
      s_warp[lane] = t;
    }
    __syncthreads();
    const unsigned long long before = s_base + (warp ? s_warp[warp - 1] : 0ull) + (run - x[3]);
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (i + e < nk) c[i + e + 1] = before + x[e];
    __syncthreads();
    if (tid == 1023) s_base = before + x[3];
    __syncthreads();
  }
}

struct VnormSampleArgs {
  const unsigned long long* cum;   // [G, nk + 1]
  int32_t* samples;                // [G, nodes, m]
  float* wlog;                     // [G, nodes, m] log2 of the weight 1 / (m p) of every draw
  Geometry g;
  uint32_t k0, k1;
};

__global__ void __launch_bounds__(256) vnorm_sample_kernel(VnormSampleArgs a) {
  const Geometry& g = a.g;
  const size_t total_draws = (size_t)g.G * g.nodes * g.m;
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= total_draws) return;
  const int jd = (int)(i % g.m);
  const int nd = (int)((i / g.m) % g.nodes);
  const int seg = (int)(i / ((size_t)g.m * g.nodes));
  const int level = g.causal ? 31 - __clz(nd + 1) : 0;
  int s, q0, k0;
  node_rows(g, level, g.causal ? nd + 1 - (1 << level) : 0, s, q0, k0);
  const Philox4 x4 = philox4x32_10((uint32_t)(jd >> 2), (uint32_t)(g.seg0 + seg), (uint32_t)nd, kDomainSamples, a.k0, a.k1);
  const uint32_t x = x4.x[jd & 3];
  const unsigned long long* c = a.cum + (size_t)seg * (g.nk + 1) + k0;     // c[l] - c[0]: weight of the node's first l keys
  const int have = min(s, g.nk - k0);                                     // keys of the node that exist
  int idx;
  float wl;
  const unsigned long long base = have > 0 ? c[0] : 0ull;
  const unsigned long long total = have > 0 ? c[have] - base : 0ull;
  if (total == 0ull) {
    idx = (int)__umulhi(x, (uint32_t)s);
    wl = g.m > 0 ? log2f((float)s / (float)g.m) : 0.f;
  } else {
    const unsigned long long target = __umul64hi((unsigned long long)x << 32, total);     // floor(x * total / 2^32)
    int lo = 0, hi = have - 1;                           // smallest l with c[l + 1] - base > target
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (c[mid + 1] - base > target) hi = mid; else lo = mid + 1;
    }
    idx = lo;
    const unsigned long long w = c[idx + 1] - c[idx];
    wl = log2f((float)total / ((float)g.m * (float)w));
  }
  a.samples[i] = idx;
  a.wlog[i] = wl;
}

}  // namespace

cudaError_t launch_vnorm_sampling(const Geometry& g, const __nv_bfloat16* v, uint32_t* wq, unsigned long long* cum, int32_t* samples,
                                  float* wlog, uint64_t seed, cudaStream_t st) {
  if (!g.sorted || g.m == 0 || g.nodes == 0) return cudaSuccess;
  const size_t rows = (size_t)g.G * g.nk;
  const size_t blocks = (rows + 255) / 256;
  if (blocks > 0x7fffffffull) return cudaErrorInvalidValue;
  if (g.d == 64) vnorm_weights_kernel<64><<<(unsigned)blocks, 256, 0, st>>>(v, wq, rows);
  else vnorm_weights_kernel<128><<<(unsigned)blocks, 256, 0, st>>>(v, wq, rows);
  vnorm_scan_kernel<<<g.G, 1024, 0, st>>>(wq, cum, g.nk);
  VnormSampleArgs a;
  a.cum = cum; a.samples = samples; a.wlog = wlog; a.g = g; a.k0 = (uint32_t)seed; a.k1 = (uint32_t)(seed >> 32);
  const size_t draws = (size_t)g.G * g.nodes * g.m;
  vnorm_sample_kernel<<<(unsigned)((draws + 255) / 256), 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hyperattn
