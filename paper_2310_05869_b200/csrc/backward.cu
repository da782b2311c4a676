// Backward pass of the HyperAttention forward map (the paper times one in Sec. 4.2 without
// writing it down): the derivative of out = rownorm(C o exp(scale Q K^T)) V with the sortLSH
// permutations and the sampled columns - hence the coefficient matrix C of Alg. 2 lines 7
// and 9 and of the causal recursion of Alg. 4 - held fixed.  With P = rownorm(C o A), which
// the forward pass's log-sum-exp gives back as P_ij = C_ij exp(s_ij - lse_i):
//     delta_i = <dO_i, O_i>
//     dV_j   += sum_i P_ij dO_i
//     dS_ij   = P_ij (<dO_i, V_j> - delta_i)
//     dQ_i   += scale sum_j dS_ij K_j,      dK_j += scale sum_i dS_ij Q_i.
// The merge of the causal recursion needs no derivative of its own: the merged output is one
// softmax over everything a row sees, so every tile of every level uses the FINAL lse and delta.
//
// First version, on the warp-level tensor-core path (mma.sync m16n8k16): one CTA per query
// tile of the forward schedule, the same row tables, S and dP like the forward's S, dQ like
// its O; P and dS are staged in shared memory so that the transposed products (dV, dK) can
// read them with ldmatrix.trans, and all three gradients are accumulated in fp32 with global
// reductions (a key tile is shared by every query tile that samples it).
#include "attn_common.cuh"

namespace hyperattn {
namespace {

constexpr int TK = 64;   // keys per tile

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void st_shared_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
// byte offset of 16-byte chunk c of row `row` in a [ROWS x 64k] bf16 tile: slabs of [ROWS x 128 B], 128-byte swizzle
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int row, int c) {
  return (uint32_t)((c >> 3) * (ROWS * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}
template <int D, int ROWS, class RowFn>
__device__ __forceinline__ void gather_tile(uint32_t dst, const __nv_bfloat16* src, RowFn rowfn, int tid) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int i = 0; i < ROWS * CPR / 256; ++i) {
    const int c = tid + i * 256;
    const int row = c / CPR, cc = c % CPR;
    const int gr = rowfn(row);
    const uint32_t d = dst + tile_off<ROWS>(row, cc);
    if (gr >= 0) cp_async16(d, src + (size_t)gr * D + cc * 8);
    else st_shared_zero16(d);
  }
}
__device__ __forceinline__ void red_add2(float* p, float x, float y) {
  atomicAdd(reinterpret_cast<float2*>(p), make_float2(x, y));
}

struct BwdArgs {
  AttnArgs a;
  const __nv_bfloat16* dout;   // [G, n, D]
  const float* lse;            // [G, n] final log-sum-exp of the forward pass (natural log)
  const float* delta;          // [G, n] <dO_i, O_i>
  float *dq, *dk, *dv;         // [G, n, D] fp32 accumulators, zeroed before the launch
  float scale;
  int table_keys;              // key columns of a node tile's row tables (block and samples, each padded to whole tiles)
};

template <int D>
struct Smem {
  static constexpr int kQ = kTileQ * D * 2;
  static constexpr int kKV = TK * D * 2;
  static constexpr int kP = kTileQ * TK * 2;
  static constexpr int kFixed = 2 * kQ + 4 * kKV + 2 * kP + kTileQ * 12;   // + 8 bytes per key column of the row tables
};

// delta_i = <dO_i, O_i>: one warp per row
template <int D, bool OUT_FP32>
__global__ void __launch_bounds__(256) delta_kernel(const __nv_bfloat16* __restrict__ dout, const void* __restrict__ out,
                                                    float* __restrict__ delta, size_t rows) {
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float acc = 0.f;
  for (int c = lane; c < D; c += 32) {
    const float o = OUT_FP32 ? reinterpret_cast<const float*>(out)[row * D + c]
                             : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(out)[row * D + c]);
    acc += o * __bfloat162float(dout[row * D + c]);
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) delta[row] = acc;
}

// (d = 64: two CTAs per SM - the legacy tensor path needs the warps to hide its latencies)
template <int D>
__global__ void __launch_bounds__(256, D == 64 ? 2 : 1) bwd_kernel(const __grid_constant__ BwdArgs b) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using SM = Smem<D>;
  const AttnArgs& a = b.a;
  uint8_t* sQ = smem;
  uint8_t* sdO = sQ + SM::kQ;
  uint8_t* sK = sdO + SM::kQ;                     // [2][TK x D]
  uint8_t* sV = sK + 2 * SM::kKV;                 // [2][TK x D]
  uint8_t* sP = sV + 2 * SM::kKV;                 // [128 x TK] bf16, P of the current key tile
  uint8_t* sdS = sP + SM::kP;                     // [128 x TK] bf16, dS of the current key tile
  int* s_qrow = reinterpret_cast<int*>(sdS + SM::kP);
  float* s_lse2 = reinterpret_cast<float*>(s_qrow + kTileQ);
  float* s_delta = s_lse2 + kTileQ;
  int* s_kidx = reinterpret_cast<int*>(s_delta + kTileQ);       // [table_keys]
  float* s_kbias = reinterpret_cast<float*>(s_kidx + b.table_keys);

  const Geometry& g = a.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const TileDesc t = decode_tile(a, blockIdx.x);
  if (t.nq <= 0) return;

  const size_t seg_row0 = (size_t)t.seg * g.n;
  const __nv_bfloat16* qs = a.q + seg_row0 * D;
  const __nv_bfloat16* ks = a.k + seg_row0 * D;
  const __nv_bfloat16* vs = a.v + seg_row0 * D;
  const __nv_bfloat16* dos = b.dout + seg_row0 * D;

  // ---- row tables (as in the forward pass) ------------------------------------------------
  int nkeys;
  if (t.mode == 1) {
    const int bpad = (g.b + TK - 1) / TK * TK, mpad = (g.m + TK - 1) / TK * TK;
    nkeys = bpad + mpad;
    const float wlog = g.m > 0 ? log2f((float)t.nk / (float)g.m) : 0.f;
    const int32_t* smp = a.samples + ((size_t)t.seg * g.nodes + t.node) * g.m;
    for (int i = tid; i < nkeys; i += 256) {
      int idx = -1; float bias = -INFINITY;
      if (i < bpad) {
        if (i < block_len(t.nk, g.b, t.beta)) { idx = t.k0 + a.perm_k[t.slice + (size_t)t.beta * g.b + i]; bias = 0.f; }
      } else if (i - bpad < g.m) {
        const int l = smp[i - bpad];
        idx = t.k0 + l;
        bias = (a.rank_k[t.slice + l] / g.b == t.beta) ? -INFINITY : wlog;
      }
      s_kidx[i] = idx; s_kbias[i] = bias;
    }
    if (tid < kTileQ) s_qrow[tid] = tid < t.nq ? t.qnode0 + a.perm_q[t.slice + t.spos0 + tid] : -1;
  } else {
    const int lim = t.causal ? min(t.nk, t.qk_off + t.nq) : t.nk;
    nkeys = (lim + TK - 1) / TK * TK;
    if (tid < kTileQ) s_qrow[tid] = tid < t.nq ? t.q0 + tid : -1;
  }
  __syncthreads();
  if (tid < kTileQ) {
    const int qr = s_qrow[tid];
    // (a padding row gets lse = +inf, so that all its weights are zero)
    s_lse2[tid] = qr >= 0 ? b.lse[seg_row0 + qr] * 1.4426950408889634f : INFINITY;
    s_delta[tid] = qr >= 0 ? b.delta[seg_row0 + qr] : 0.f;
  }

  const uint32_t uQ = smem_u32(sQ), udO = smem_u32(sdO), uK = smem_u32(sK), uV = smem_u32(sV);
  const uint32_t uP = smem_u32(sP), udS = smem_u32(sdS);
  auto qrow_fn = [&](int r) { return s_qrow[r]; };
  auto krow_of = [&](int i) {          // segment-relative key row of key column i, -1: padding
    if (t.mode == 1) return s_kidx[i];
    return i < t.nk ? t.k0 + i : -1;
  };
  auto load_kv = [&](int kt, int stage) {
    auto krow_fn = [&](int r) { return krow_of(kt * TK + r); };
    gather_tile<D, TK>(uK + stage * SM::kKV, ks, krow_fn, tid);
    gather_tile<D, TK>(uV + stage * SM::kKV, vs, krow_fn, tid);
  };
  gather_tile<D, kTileQ>(uQ, qs, qrow_fn, tid);
  gather_tile<D, kTileQ>(udO, dos, qrow_fn, tid);
  const int ntiles = nkeys / TK;
  load_kv(0, 0);
  cp_async_commit();

  constexpr int KS = D / 16, NO = D / 8;
  float dq[NO][4];
#pragma unroll
  for (int i = 0; i < NO; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }
  const int r_lo = warp * 16 + gid, r_hi = r_lo + 8;      // this lane's two query rows in the tile

  for (int kt = 0; kt < ntiles; ++kt) {
    const int stage = kt & 1;
    if (kt + 1 < ntiles) load_kv(kt + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    const uint32_t kb = uK + stage * SM::kKV, vb = uV + stage * SM::kKV;
    // S = Q K^T and dP = dO V^T : 16 x 64 per warp each
    float sc[TK / 8][4], dp[TK / 8][4];
#pragma unroll
    for (int i = 0; i < TK / 8; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; dp[i][0] = dp[i][1] = dp[i][2] = dp[i][3] = 0.f; }
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      uint32_t qf[4], df[4];
      ldmatrix_x4(qf, uQ + tile_off<kTileQ>(warp * 16 + (lane & 15), 2 * s + (lane >> 4)));
      ldmatrix_x4(df, udO + tile_off<kTileQ>(warp * 16 + (lane & 15), 2 * s + (lane >> 4)));
#pragma unroll
      for (int np = 0; np < TK / 16; ++np) {
        uint32_t bf[4];
        const uint32_t koff = tile_off<TK>(np * 16 + (lane & 7) + ((lane >> 4) << 3), 2 * s + ((lane >> 3) & 1));
        ldmatrix_x4(bf, kb + koff);
        mma_16816(sc[2 * np], qf, bf[0], bf[1]);
        mma_16816(sc[2 * np + 1], qf, bf[2], bf[3]);
        ldmatrix_x4(bf, vb + koff);
        mma_16816(dp[2 * np], df, bf[0], bf[1]);
        mma_16816(dp[2 * np + 1], df, bf[2], bf[3]);
      }
    }
    // P = C o exp(s - lse) (the coefficient is an additive bias on the log2 logit), dS = P (dP - delta)
    uint32_t dsf[TK / 16][4];
#pragma unroll
    for (int nt = 0; nt < TK / 8; ++nt) {
      float p[4], ds[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = kt * TK + nt * 8 + 2 * tig + (e & 1);
        const int row = (e & 2) ? r_hi : r_lo;
        float x = sc[nt][e] * a.scale_log2;
        if (t.mode == 1) x += s_kbias[col];
        else if (col >= t.nk || (t.causal && col > t.qk_off + row)) x = -INFINITY;
        p[e] = exp2f(x - s_lse2[row]);
        ds[e] = p[e] * (dp[nt][e] - s_delta[row]);
      }
      const uint32_t p01 = pack2(p[0], p[1]), p23 = pack2(p[2], p[3]);
      const uint32_t d01 = pack2(ds[0], ds[1]), d23 = pack2(ds[2], ds[3]);
      dsf[nt >> 1][(nt & 1) * 2] = d01;
      dsf[nt >> 1][(nt & 1) * 2 + 1] = d23;
      // staged [query row][key column] for the transposed products
      const uint32_t o_lo = tile_off<kTileQ>(r_lo, nt) + 4 * tig, o_hi = tile_off<kTileQ>(r_hi, nt) + 4 * tig;
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(uP + o_lo), "r"(p01));
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(uP + o_hi), "r"(p23));
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(udS + o_lo), "r"(d01));
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(udS + o_hi), "r"(d23));
    }
    // dQ += dS K
#pragma unroll
    for (int kk = 0; kk < TK / 16; ++kk) {
#pragma unroll
      for (int dpi = 0; dpi < NO / 2; ++dpi) {
        uint32_t bf[4];
        ldmatrix_x4_trans(bf, kb + tile_off<TK>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * dpi + (lane >> 4)));
        mma_16816(dq[2 * dpi], dsf[kk], bf[0], bf[1]);
        mma_16816(dq[2 * dpi + 1], dsf[kk], bf[2], bf[3]);
      }
    }
    __syncthreads();   // P and dS of all 128 rows are staged
    // Transposed products over the 128 query rows: warps 0-3 dV = P^T dO, warps 4-7 dK = dS^T Q,
    // 16 keys of the tile per warp.
    {
      const int w4 = warp & 3;
      const uint32_t uA = warp < 4 ? uP : udS;             // [query][key], read transposed
      const uint32_t uB = warp < 4 ? udO : uQ;             // [query][d]
      float acc[NO][4];
#pragma unroll
      for (int i = 0; i < NO; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
#pragma unroll
      for (int kq = 0; kq < kTileQ / 16; ++kq) {
        uint32_t af[4];
        // A (16 keys x 16 queries) = transpose of the staged block: matrix (mi, ki) comes from query rows
        // 16 kq + 8 ki .., key chunk 2 w4 + mi
        ldmatrix_x4_trans(af, uA + tile_off<kTileQ>(kq * 16 + ((lane >> 4) << 3) + (lane & 7), 2 * w4 + ((lane >> 3) & 1)));
#pragma unroll
        for (int dpi = 0; dpi < NO / 2; ++dpi) {
          uint32_t bf[4];
          ldmatrix_x4_trans(bf, uB + tile_off<kTileQ>(kq * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * dpi + (lane >> 4)));
          mma_16816(acc[2 * dpi], af, bf[0], bf[1]);
          mma_16816(acc[2 * dpi + 1], af, bf[2], bf[3]);
        }
      }
      const float f = warp < 4 ? 1.f : b.scale;
      float* dst = warp < 4 ? b.dv : b.dk;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int kr = krow_of(kt * TK + w4 * 16 + gid + 8 * h);
        if (kr < 0) continue;
        float* rowp = dst + (seg_row0 + kr) * D;
#pragma unroll
        for (int i = 0; i < NO; ++i) red_add2(rowp + i * 8 + 2 * tig, acc[i][2 * h] * f, acc[i][2 * h + 1] * f);
      }
    }
    __syncthreads();   // everyone is done with this stage and with the staged P / dS
  }
  cp_async_wait<0>();

  // ---- dQ: rows back to their original places (a row collects from every level it appears in) ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int qr = s_qrow[h ? r_hi : r_lo];
    if (qr < 0) continue;
    float* rowp = b.dq + (seg_row0 + qr) * D;
#pragma unroll
    for (int i = 0; i < NO; ++i) red_add2(rowp + i * 8 + 2 * tig, dq[i][2 * h] * b.scale, dq[i][2 * h + 1] * b.scale);
  }
}

__global__ void to_bf16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, size_t count4) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 v = src[i];
    dst[i] = make_uint2(pack2(v.x, v.y), pack2(v.z, v.w));
  }
}

}  // namespace

// a: the forward schedule (tile list, permutations, samples); dq/dk/dv accumulators must be zero
cudaError_t launch_backward(const AttnArgs& a, const void* out, int out_fp32, const float* lse, const void* dout,
                            float* delta, float* dq, float* dk, float* dv, float scale, cudaStream_t st) {
  const size_t rows = (size_t)a.g.G * a.g.n;
  const __nv_bfloat16* d16 = reinterpret_cast<const __nv_bfloat16*>(dout);
  const int dgrid = (int)((rows + 7) / 8);
  if (a.g.d == 64) {
    if (out_fp32) delta_kernel<64, true><<<dgrid, 256, 0, st>>>(d16, out, delta, rows);
    else delta_kernel<64, false><<<dgrid, 256, 0, st>>>(d16, out, delta, rows);
  } else {
    if (out_fp32) delta_kernel<128, true><<<dgrid, 256, 0, st>>>(d16, out, delta, rows);
    else delta_kernel<128, false><<<dgrid, 256, 0, st>>>(d16, out, delta, rows);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || a.total_tiles == 0) return e;
  BwdArgs b;
  b.a = a; b.dout = d16; b.lse = lse; b.delta = delta; b.dq = dq; b.dk = dk; b.dv = dv; b.scale = scale;
  b.table_keys = a.g.sorted ? (a.g.b + TK - 1) / TK * TK + (a.g.m + TK - 1) / TK * TK : 0;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e2 = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes + kMaxNodeKeys * 8);
    if (e2 != cudaSuccess) return e2;
    kernel<<<a.total_tiles, 256, smem_bytes + b.table_keys * 8, st>>>(b);
    return cudaGetLastError();
  };
  if (a.g.d == 64) return go(bwd_kernel<64>, Smem<64>::kFixed);
  return go(bwd_kernel<128>, Smem<128>::kFixed);
}

cudaError_t launch_to_bf16(const float* src, void* dst, size_t count, cudaStream_t st) {
  const size_t count4 = count / 4;
  int blocks = (int)((count4 + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  to_bf16_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(dst), count4);
  return cudaGetLastError();
}

}  // namespace hyperattn
