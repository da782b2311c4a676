// The quantity the paper's guarantee is stated in (Theorem 1, measured in Sec. 4.3):
//     alpha = n * max_j || D^-1 A e_j ||_2^2,
// n times the largest squared column norm of the exact softmax matrix D^-1 A, A = exp(scale Q K^T)
// (with the causal mask M^C when asked for; Sec. 4.3 leaves out the first columns of causal models,
// which hold heavy entries: skip_cols).  A diagnostic, not part of the forward pass: it costs the
// full n x n_k matrix twice.  Three small kernels on the warp-level tensor cores (mma.sync
// m16n8k16; 16 query rows per CTA against every key):
//   1. row pass:     lse2_i = log2 sum_j exp2(s_ij)                  (s in the scaled base-2 domain)
//   2. column pass:  c_j += sum_i exp2(2 (s_ij - lse2_i))             (fp32 atomics, one per 16 rows and key)
//   3. maximum over j >= skip_cols, times n.
#include "../../include/hyperattn.h"
#include "common.cuh"

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
__device__ __forceinline__ void lse_merge(float& m, float& l, float m2, float l2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) return;
  l = l * ex2f(m - mn) + l2 * ex2f(m2 - mn);
  m = mn;
}

struct AlphaArgs {
  const __nv_bfloat16 *q, *k;
  int G, n, nk, causal, skip_cols;
  float scale_log2;
  float* lse2;     // [G, n]
  float* colsq;    // [G, nk], zeroed before the column pass
  float* alpha;    // [G]
};

// PASS 0: row pass, PASS 1: column pass.  One CTA: 16 query rows of one segment; the 8 warps split the keys.
template <int D, int PASS>
__global__ void __launch_bounds__(256) alpha_rows_kernel(const __grid_constant__ AlphaArgs a) {
  constexpr int KS = D / 16, CPL = D / 32;
  constexpr int U = D == 64 ? 4 : 2;
  __shared__ float s_m[8][16], s_l[8][16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
  const int groups = (a.n + 15) / 16;
  const int rg = blockIdx.x % groups, seg = blockIdx.x / groups;
  int row[2];
  float lse_r[2] = {0.f, 0.f};
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    row[r] = rg * 16 + gid + 8 * r;
    if (row[r] >= a.n) row[r] = -1;
    if (PASS == 1 && row[r] >= 0) lse_r[r] = a.lse2[(size_t)seg * a.n + row[r]];
  }
  // (same coordinate-to-slot assignment for rows and keys, so that every lane fetches 16-byte pieces)
  uint32_t af[KS][4];
  {
    const char* qb = reinterpret_cast<const char*>(a.q) + (size_t)seg * a.n * (D * 2);
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
  const char* kb = reinterpret_cast<const char*>(a.k) + (size_t)seg * a.nk * (D * 2);
  float m2[2] = {-INFINITY, -INFINITY}, l2[2] = {0.f, 0.f};
  // causal: keys beyond the group's last row are masked for every row of the group
  const int klim = a.causal ? min(a.nk, rg * 16 + 16) : a.nk;
  const int nblocks = (klim + 7) / 8;
  for (int nb0 = warp * U; nb0 < nblocks; nb0 += 8 * U) {
    uint4 vk[U][CPL];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int key = (nb0 + u) * 8 + gid;
#pragma unroll
      for (int h = 0; h < CPL; ++h)
        vk[u][h] = key < klim ? *reinterpret_cast<const uint4*>(kb + (size_t)key * (D * 2) + (tig + 4 * h) * 16) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int st = 0; st < KS; ++st)
        mma_16816(c, af[st], (st & 1) ? vk[u][st >> 1].z : vk[u][st >> 1].x, (st & 1) ? vk[u][st >> 1].w : vk[u][st >> 1].y);
      const int col = (nb0 + u) * 8 + 2 * tig;
      float sq[2] = {0.f, 0.f};                           // column pass: this lane's share of the two columns
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        float x[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool vis = row[r] >= 0 && col + e < a.nk && (!a.causal || col + e <= row[r]);
          x[e] = vis ? c[2 * r + e] * a.scale_log2 : -INFINITY;
        }
        if (PASS == 0) {
          const float mn = fmaxf(m2[r], fmaxf(x[0], x[1]));
          if (mn > -INFINITY) {
            l2[r] = l2[r] * ex2f(m2[r] - mn) + ex2f(x[0] - mn) + ex2f(x[1] - mn);
            m2[r] = mn;
          }
        } else {
          sq[0] += ex2f(2.f * (x[0] - lse_r[r]));
          sq[1] += ex2f(2.f * (x[1] - lse_r[r]));
        }
      }
      if (PASS == 1) {
        // the eight row pairs of the group (lanes with the same tig) add up, then one atomic per column
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
          sq[0] += __shfl_xor_sync(0xffffffffu, sq[0], o);
          sq[1] += __shfl_xor_sync(0xffffffffu, sq[1], o);
        }
        if (gid == 0) {
          if (col < a.nk && sq[0] > 0.f) atomicAdd(a.colsq + (size_t)seg * a.nk + col, sq[0]);
          if (col + 1 < a.nk && sq[1] > 0.f) atomicAdd(a.colsq + (size_t)seg * a.nk + col + 1, sq[1]);
        }
      }
    }
  }
  if (PASS == 0) {
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
    if (warp == 0 && lane < 16 && rg * 16 + lane < a.n) {
      float m = s_m[0][lane], l = s_l[0][lane];
#pragma unroll
      for (int w = 1; w < 8; ++w) lse_merge(m, l, s_m[w][lane], s_l[w][lane]);
      a.lse2[(size_t)seg * a.n + rg * 16 + lane] = m + log2f(l);
    }
  }
}

__global__ void __launch_bounds__(256) alpha_max_kernel(AlphaArgs a) {
  __shared__ float s_best[8];
  const int seg = blockIdx.x;
  float best = 0.f;
  for (int jc = a.skip_cols + threadIdx.x; jc < a.nk; jc += 256) best = fmaxf(best, a.colsq[(size_t)seg * a.nk + jc]);
#pragma unroll
  for (int o = 16; o; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
  if ((threadIdx.x & 31) == 0) s_best[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) best = fmaxf(best, s_best[w]);
    a.alpha[seg] = (float)a.n * best;
  }
}

}  // namespace
}  // namespace hyperattn

using namespace hyperattn;

extern "C" int hyperattn_alpha_workspace_bytes(int B, int H, int n, int n_k, size_t* bytes) {
  if (!bytes || B <= 0 || H <= 0 || n <= 0 || n_k < 0) return HYPERATTN_INVALID_ARGUMENT;
  const size_t G = (size_t)B * H;
  *bytes = G * ((size_t)n + (size_t)(n_k ? n_k : n)) * 4 + 512;
  return HYPERATTN_OK;
}

extern "C" int hyperattn_alpha(const void* q, const void* k, int B, int H, int n, int n_k, int d, float softmax_scale,
                               int causal, int skip_cols, float* alpha, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !k || !alpha || !workspace) return HYPERATTN_INVALID_ARGUMENT;
  if (B <= 0 || H <= 0 || n <= 0 || n_k < 0 || skip_cols < 0) return HYPERATTN_INVALID_ARGUMENT;
  if (d != 64 && d != 128) return HYPERATTN_UNSUPPORTED_SHAPE;
  const int nk = n_k ? n_k : n;
  if (causal && nk != n) return HYPERATTN_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(k) & 15) || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return HYPERATTN_MISALIGNED;
  size_t need = 0;
  hyperattn_alpha_workspace_bytes(B, H, n, nk, &need);
  if (workspace_bytes < need) return HYPERATTN_WORKSPACE_TOO_SMALL;
  const size_t G = (size_t)B * H;
  const long long grid = (long long)G * ((n + 15) / 16);
  if (grid > 0x7fffffffLL || G > 0x7fffffffull) return HYPERATTN_UNSUPPORTED_SHAPE;
  AlphaArgs a;
  a.q = reinterpret_cast<const __nv_bfloat16*>(q); a.k = reinterpret_cast<const __nv_bfloat16*>(k);
  a.G = (int)G; a.n = n; a.nk = nk; a.causal = causal != 0; a.skip_cols = skip_cols;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.f / sqrtf((float)d);
  a.scale_log2 = scale * 1.4426950408889634f;
  char* base = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(workspace) + 255) / 256 * 256);
  a.lse2 = reinterpret_cast<float*>(base);
  a.colsq = a.lse2 + G * (size_t)n;
  a.alpha = alpha;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(a.colsq, 0, G * (size_t)nk * 4, st) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (d == 64) {
    alpha_rows_kernel<64, 0><<<(unsigned)grid, 256, 0, st>>>(a);
    alpha_rows_kernel<64, 1><<<(unsigned)grid, 256, 0, st>>>(a);
  } else {
    alpha_rows_kernel<128, 0><<<(unsigned)grid, 256, 0, st>>>(a);
    alpha_rows_kernel<128, 1><<<(unsigned)grid, 256, 0, st>>>(a);
  }
  alpha_max_kernel<<<(unsigned)G, 256, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? HYPERATTN_OK : HYPERATTN_CUDA_ERROR;
}
