// Attention tiles on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32
// accumulate): block-diagonal part (Sec. 4), sampled residual (Alg. 2 line 7) and exact
// causal leaves (Sec. 3.1) with one online-softmax loop.  Rows of Q, K, V are gathered
// straight from their original places through the sortLSH permutations with 16-byte
// cp.async copies into 128-byte-swizzled shared memory, so no permuted copy of the inputs
// is ever written to HBM.
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

// byte offset of 16-byte chunk `c` (0 .. D/8-1) of row `row` in a [ROWS x D] bf16 tile stored
// as D/64 slabs of [ROWS x 128 B] with the 128-byte swizzle (chunk ^= row & 7)
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int row, int c) {
  return (uint32_t)((c >> 3) * (ROWS * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

// gather ROWS rows (index -1 = zero row) of a [*, D] bf16 tensor into a swizzled tile
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

template <int D, bool SPLIT>
struct Smem {
  static constexpr int kQ = kTileQ * D * 2;
  static constexpr int kKV = TK * D * 2;
  static constexpr int kTotal = (SPLIT ? 2 : 1) * kQ + (SPLIT ? 6 : 4) * kKV + kMaxNodeKeys * 8 + kTileQ * 4;
};

// SPLIT: the inputs were fp32 and arrive as two bf16 terms (x = hi + lo up to 2^-17 relative);
// the logits use Q_hi K_hi + Q_lo K_hi + Q_hi K_lo so that they keep fp32-like accuracy.
template <int D, bool SPLIT>
__global__ void __launch_bounds__(256, 1) attn_mma_kernel(const __grid_constant__ AttnArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using SM = Smem<D, SPLIT>;
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + SM::kQ;                      // [2][TK x D]
  uint8_t* sV = sK + 2 * SM::kKV;                 // [2][TK x D]
  uint8_t* sQl = sV + 2 * SM::kKV;                // SPLIT only
  uint8_t* sKl = sQl + (SPLIT ? SM::kQ : 0);      // SPLIT only: [2][TK x D]
  int* s_kidx = reinterpret_cast<int*>(sKl + (SPLIT ? 2 * SM::kKV : 0));
  float* s_kbias = reinterpret_cast<float*>(s_kidx + kMaxNodeKeys);
  int* s_qrow = reinterpret_cast<int*>(s_kbias + kMaxNodeKeys);

  const Geometry& g = a.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const TileDesc t = decode_tile(a, blockIdx.x);
  if (t.nq <= 0) return;                          // (a tile of the schedule whose rows do not exist)

  const __nv_bfloat16* qs = a.q + (size_t)t.seg * g.n * D;
  const __nv_bfloat16* ks = a.k + (size_t)t.seg * g.nk * D;
  const __nv_bfloat16* vs = a.v + (size_t)t.seg * g.nk * D;

  // ---- row tables ---------------------------------------------------------------------
  int nkeys;  // padded number of key columns visited
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

  const uint32_t uQ = smem_u32(sQ), uK = smem_u32(sK), uV = smem_u32(sV);
  const uint32_t uQl = smem_u32(sQl), uKl = smem_u32(sKl);
  const __nv_bfloat16* qls = a.q_lo + (size_t)t.seg * g.n * D;
  const __nv_bfloat16* kls = a.k_lo + (size_t)t.seg * g.nk * D;
  auto qrow_fn = [&](int r) { return s_qrow[r]; };
  auto load_kv = [&](int kt, int stage) {
    auto krow_fn = [&](int r) {
      const int i = kt * TK + r;
      if (t.mode == 1) return s_kidx[i];
      return i < t.nk ? t.k0 + i : -1;
    };
    gather_tile<D, TK>(uK + stage * SM::kKV, ks, krow_fn, tid);
    gather_tile<D, TK>(uV + stage * SM::kKV, vs, krow_fn, tid);
    if constexpr (SPLIT) gather_tile<D, TK>(uKl + stage * SM::kKV, kls, krow_fn, tid);
  };

  gather_tile<D, kTileQ>(uQ, qs, qrow_fn, tid);
  if constexpr (SPLIT) gather_tile<D, kTileQ>(uQl, qls, qrow_fn, tid);
  const int ntiles = nkeys / TK;
  load_kv(0, 0);
  cp_async_commit();

  // ---- per-warp state: 16 query rows ----------------------------------------------------
  constexpr int KS = D / 16, NO = D / 8;
  uint32_t qf[SPLIT ? 1 : KS][4];
  float o[NO][4];
#pragma unroll
  for (int i = 0; i < NO; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const int r_lo = warp * 16 + gid, r_hi = r_lo + 8;      // this lane's two rows in the tile

  for (int kt = 0; kt < ntiles; ++kt) {
    const int stage = kt & 1;
    if (kt + 1 < ntiles) load_kv(kt + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if constexpr (!SPLIT) {
      if (kt == 0) {
#pragma unroll
        for (int s = 0; s < KS; ++s)
          ldmatrix_x4(qf[s], uQ + tile_off<kTileQ>(warp * 16 + (lane & 15), 2 * s + (lane >> 4)));
      }
    }
    // S = Q K^T : 16 x 64 per warp
    float sc[TK / 8][4];
#pragma unroll
    for (int i = 0; i < TK / 8; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
    const uint32_t kb = uK + stage * SM::kKV;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      uint32_t ql[4];
      if constexpr (SPLIT) {
        ldmatrix_x4(qf[0], uQ + tile_off<kTileQ>(warp * 16 + (lane & 15), 2 * s + (lane >> 4)));
        ldmatrix_x4(ql, uQl + tile_off<kTileQ>(warp * 16 + (lane & 15), 2 * s + (lane >> 4)));
      }
      const uint32_t(&qh)[4] = qf[SPLIT ? 0 : s];
#pragma unroll
      for (int np = 0; np < TK / 16; ++np) {
        uint32_t bf[4];
        const uint32_t koff = tile_off<TK>(np * 16 + (lane & 7) + ((lane >> 4) << 3), 2 * s + ((lane >> 3) & 1));
        if constexpr (SPLIT) {
          uint32_t bl[4];
          ldmatrix_x4(bl, uKl + stage * SM::kKV + koff);
          mma_16816(sc[2 * np], qh, bl[0], bl[1]);
          mma_16816(sc[2 * np + 1], qh, bl[2], bl[3]);
        }
        ldmatrix_x4(bf, kb + koff);
        if constexpr (SPLIT) {
          mma_16816(sc[2 * np], ql, bf[0], bf[1]);
          mma_16816(sc[2 * np + 1], ql, bf[2], bf[3]);
        }
        mma_16816(sc[2 * np], qh, bf[0], bf[1]);
        mma_16816(sc[2 * np + 1], qh, bf[2], bf[3]);
      }
    }
    // logits in log2 units, masks
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < TK / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = kt * TK + nt * 8 + 2 * tig + (e & 1);
        const int row = (e & 2) ? r_hi : r_lo;
        float x = sc[nt][e] * a.scale_log2;
        if (t.mode == 1) x += s_kbias[col];
        else if (col >= t.nk || (t.causal && col > t.qk_off + row)) x = -INFINITY;
        sc[nt][e] = x;
        mx[e >> 1] = fmaxf(mx[e >> 1], x);
      }
    }
    float alpha[2], muse[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float mnew = fmaxf(mrow[h], mx[h]);
      muse[h] = mnew == -INFINITY ? 0.f : mnew;
      alpha[h] = exp2f(mrow[h] - muse[h]);
      mrow[h] = mnew;
      lrow[h] *= alpha[h];
    }
#pragma unroll
    for (int i = 0; i < NO; ++i) { o[i][0] *= alpha[0]; o[i][1] *= alpha[0]; o[i][2] *= alpha[1]; o[i][3] *= alpha[1]; }
    uint32_t pf[TK / 16][4];
#pragma unroll
    for (int nt = 0; nt < TK / 8; ++nt) {
      const float p0 = exp2f(sc[nt][0] - muse[0]), p1 = exp2f(sc[nt][1] - muse[0]);
      const float p2 = exp2f(sc[nt][2] - muse[1]), p3 = exp2f(sc[nt][3] - muse[1]);
      lrow[0] += p0 + p1; lrow[1] += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2] = pack2(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack2(p2, p3);
    }
    // O += P V
    const uint32_t vb = uV + stage * SM::kKV;
#pragma unroll
    for (int kk = 0; kk < TK / 16; ++kk) {
#pragma unroll
      for (int dp = 0; dp < NO / 2; ++dp) {
        uint32_t bf[4];
        ldmatrix_x4_trans(bf, vb + tile_off<TK>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * dp + (lane >> 4)));
        mma_16816(o[2 * dp], pf[kk], bf[0], bf[1]);
        mma_16816(o[2 * dp + 1], pf[kk], bf[2], bf[3]);
      }
    }
    __syncthreads();   // everyone is done with this stage before it is refilled
  }
  cp_async_wait<0>();

  // ---- epilogue: normalise, log-sum-exp, scatter to the rows' original places -----------
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = h ? r_hi : r_lo;
    const int qr = s_qrow[row];
    if (qr < 0) continue;
    const float inv = 1.f / lrow[h];
    const float lse = (mrow[h] + log2f(lrow[h])) * 0.69314718055994531f;
    const size_t orow = t.orow_base + (size_t)(qr + t.odelta);
    if (t.partial) {
      float* dst = reinterpret_cast<float*>(a.part_o) + orow * D;     // (this path keeps fp32 partials)
#pragma unroll
      for (int i = 0; i < NO; ++i)
        *reinterpret_cast<float2*>(dst + i * 8 + 2 * tig) = make_float2(o[i][2 * h] * inv, o[i][2 * h + 1] * inv);
      if (tig == 0) a.part_lse[orow] = lse;
    } else {
      if (a.out_fp32) {
        float* dst = reinterpret_cast<float*>(a.out) + orow * D;
#pragma unroll
        for (int i = 0; i < NO; ++i)
          *reinterpret_cast<float2*>(dst + i * 8 + 2 * tig) = make_float2(o[i][2 * h] * inv, o[i][2 * h + 1] * inv);
      } else {
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.out) + orow * D;
#pragma unroll
        for (int i = 0; i < NO; ++i)
          *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * tig) = pack2(o[i][2 * h] * inv, o[i][2 * h + 1] * inv);
      }
      if (tig == 0) a.lse[orow] = lse;
    }
  }
}

}  // namespace

cudaError_t launch_attention_mma(const AttnArgs& a, cudaStream_t st) {
  if (a.total_tiles == 0) return cudaSuccess;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    kernel<<<a.total_tiles, 256, smem_bytes, st>>>(a);
    return cudaGetLastError();
  };
  const bool split = a.q_lo != nullptr;
  if (a.g.d == 64) return split ? go(attn_mma_kernel<64, true>, Smem<64, true>::kTotal) : go(attn_mma_kernel<64, false>, Smem<64, false>::kTotal);
  return split ? go(attn_mma_kernel<128, true>, Smem<128, true>::kTotal) : go(attn_mma_kernel<128, false>, Smem<128, false>::kTotal);
}

}  // namespace hyperattn
