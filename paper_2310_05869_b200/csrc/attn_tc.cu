// Attention tiles on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 inputs.
//
// One CTA owns one tile of 128 query rows (see attn_common.cuh for the two tile kinds) and
// walks over its key tiles of 128 keys:
//     S = Q K^T          tcgen05.mma, operands in 128B-swizzled shared memory, S in TMEM
//     P = exp2(S*c + bias - m)   softmax warps: one thread per query row (TMEM lane),
//                                P written back to TMEM as bf16 over the columns of S
//     O += P V           tcgen05.mma with P read from TMEM, V MN-major in shared memory
// which covers the block-diagonal part (Sec. 4), the sampled residual with weight N/m
// (Alg. 2 line 7) and the exact causal leaves (Sec. 3.1) in one loop.  The running row
// maximum is only moved when it grows by more than 2^8 (the accumulators absorb the
// rest), so O is rarely rescaled.  Rows of Q, K, V are gathered from their original places
// through the sortLSH permutations by three loader warps with 16-byte cp.async copies;
// nothing permuted is ever written to HBM.
//
// Warp roles (256 threads): warps 0-3 softmax + epilogue, warp 4 MMA issue + TMEM
// allocation, warps 5-7 loaders.  Two CTAs share an SM (256 TMEM columns each), so one
// CTA's softmax overlaps the other's MMAs.  Every mbarrier wait is bounded: on a timeout
// the CTA raises the device status word, drains its copies, frees its TMEM and returns.
#include "attn_common.cuh"

namespace hyperattn {
namespace {

constexpr int TK = 128;                 // keys per tile
constexpr int kLoaderThreads = 96;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every mbarrier wait gives up after 2 s
constexpr float kRescaleThreshold = 8.f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ---------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// returns false when the wait gave up (timeout or another thread aborted)
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  atomicExch(status, 1);
  return false;
}

// ---- tcgen05 ----------------------------------------------------------------------------
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of sm_100
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
               ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
               "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                 "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                 "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

// ---- copies -----------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void st_shared_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_le(int n) {   // wait until at most n groups are pending
  switch (n) {
    case 0: asm volatile("cp.async.wait_group 0;\n" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;\n" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 2;\n" ::: "memory"); break;
  }
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// byte offset of 16-byte chunk c of row `row` in a [128 x D] bf16 tile: D/64 slabs of
// [128 rows x 128 B], 128-byte swizzle inside each slab (the canonical tcgen05 layout)
__device__ __forceinline__ uint32_t tile_off(int row, int c) {
  return (uint32_t)((c >> 3) * (128 * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

template <int D>
struct Cfg {
  static constexpr int NS = (D == 64) ? 2 : 1;        // K and V stages
  static constexpr int kTile = 128 * D * 2;           // bytes of one 128-row tile
  static constexpr int kOffQ = 0;
  static constexpr int kOffK = kTile;
  static constexpr int kOffV = kOffK + NS * kTile;
  static constexpr int kOffIdx = kOffV + NS * kTile;  // int   [kMaxNodeKeys]
  static constexpr int kOffBias = kOffIdx + kMaxNodeKeys * 4;
  static constexpr int kOffQrow = kOffBias + kMaxNodeKeys * 4;    // int [128]
  static constexpr int kOffFlag = kOffQrow + 128 * 4;             // int [kMaxNodeKeys / TK] per-tile "needs table"
  static constexpr int kOffBar = kOffFlag + 64;                   // mbarriers
  static constexpr int kNumBar = 4 + 4 * NS;
  static constexpr int kOffMisc = kOffBar + 8 * kNumBar;          // tmem slot, abort flag
  static constexpr int kTotal = kOffMisc + 16;
  static constexpr int kTmemCols = 256;
  static constexpr int kColS = 0, kColO = 128;
};

template <int D>
__global__ void __launch_bounds__(256, 2) attn_tc_kernel(const __grid_constant__ AttnArgs a, int* status) {
  using C = Cfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  int* s_kidx = reinterpret_cast<int*>(smem + C::kOffIdx);
  float* s_kbias = reinterpret_cast<float*>(smem + C::kOffBias);
  int* s_qrow = reinterpret_cast<int*>(smem + C::kOffQrow);
  int* s_flag = reinterpret_cast<int*>(smem + C::kOffFlag);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);

  const uint32_t ubase = smem_u32(smem);
  const uint32_t bar0 = ubase + C::kOffBar;
  // barrier ids
  const uint32_t bar_q = bar0, bar_s = bar0 + 8, bar_p = bar0 + 16, bar_o = bar0 + 24;
  auto bar_kfull = [&](int s) { return bar0 + 32 + 8 * s; };
  auto bar_kempty = [&](int s) { return bar0 + 32 + 8 * (C::NS + s); };
  auto bar_vfull = [&](int s) { return bar0 + 32 + 8 * (2 * C::NS + s); };
  auto bar_vempty = [&](int s) { return bar0 + 32 + 8 * (3 * C::NS + s); };

  const Geometry& g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const TileDesc t = decode_tile(a, blockIdx.x);

  // A CTA of a launch in which some wait already timed out returns at once (nothing allocated
  // yet), so a stuck launch drains quickly instead of timing out tile after tile.
  if (tid == 0) *s_abort = *reinterpret_cast<volatile int*>(status);
  __syncthreads();
  if (*s_abort) return;
  __syncthreads();

  // ---- setup: barriers, TMEM, row tables ----------------------------------------------------
  if (tid == 0) {
    mbar_init(bar_q, kLoaderThreads);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 128);
    mbar_init(bar_o, 1);
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(bar_kfull(s), kLoaderThreads);
      mbar_init(bar_vfull(s), kLoaderThreads);
      mbar_init(bar_kempty(s), 1);
      mbar_init(bar_vempty(s), 1);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kMaxNodeKeys / TK) s_flag[tid] = 0;
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  __syncthreads();

  int nkeys;         // padded number of key columns visited
  float wlog = 0.f;  // log2(N/m): weight of a sampled column
  int bpad = 0;
  if (t.mode == 1) {
    bpad = (g.b + TK - 1) / TK * TK;
    const int mpad = (g.m + TK - 1) / TK * TK;
    nkeys = bpad + mpad;
    wlog = g.m > 0 ? log2f((float)t.nk / (float)g.m) : 0.f;
    const int32_t* smp = a.samples + ((size_t)t.seg * g.nodes + t.node) * g.m;
    for (int i = tid; i < nkeys; i += 256) {
      int idx = -1;
      float bias = -INFINITY;
      bool plain = false;      // entry equals the uniform value of its tile
      if (i < bpad) {
        if (i < g.b) { idx = t.k0 + a.perm_k[t.slice + (size_t)t.beta * g.b + i]; bias = 0.f; plain = true; }
      } else if (i - bpad < g.m) {
        const int l = smp[i - bpad];
        idx = t.k0 + l;
        if (a.rank_k[t.slice + l] / g.b != t.beta) { bias = wlog; plain = true; }
      }
      s_kidx[i] = idx;
      s_kbias[i] = bias;
      if (!plain) s_flag[i / TK] = 1;
    }
    if (tid < kTileQ) s_qrow[tid] = tid < t.nq ? t.qnode0 + a.perm_q[t.slice + t.spos0 + tid] : -1;
  } else {
    const int lim = t.causal ? min(t.nk, t.qk_off + t.nq) : t.nk;
    nkeys = (lim + TK - 1) / TK * TK;
    if (tid < kTileQ) s_qrow[tid] = tid < t.nq ? t.q0 + tid : -1;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const int ntiles = nkeys / TK;

  if (warp < 4) {
    // =========================== softmax + epilogue: thread = query row ======================
    const int row = tid;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < ntiles && ok; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s, j & 1, s_abort, status));   // warp-uniform: TMEM ops below are .aligned
      if (!ok) break;
      tc_fence_after();
      // per-tile mask kind (uniform over the CTA)
      bool table = false, dense_mask = false;
      float ubias = 0.f;
      if (t.mode == 1) {
        table = s_flag[j] != 0;
        ubias = (j * TK < bpad) ? 0.f : wlog;
      } else {
        dense_mask = (j * TK + TK > t.nk) || (t.causal && j * TK + TK - 1 > t.qk_off);
      }
      const int climit = t.mode == 1 ? 0 : (t.causal ? min(t.nk - 1, t.qk_off + row) : t.nk - 1);   // last visible column
      // pass 1: row maximum of the tile
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < TK / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + C::kColS + c * 32, r);
        if (table) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fmaf(__uint_as_float(r[i]), a.scale_log2, s_kbias[j * TK + c * 32 + i]));
        } else if (dense_mask) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (j * TK + c * 32 + i <= climit) mx = fmaxf(mx, __uint_as_float(r[i]) * a.scale_log2);
        } else {
          float raw = -INFINITY;
#pragma unroll
          for (int i = 0; i < 32; ++i) raw = fmaxf(raw, __uint_as_float(r[i]));
          mx = fmaxf(mx, fmaf(raw, a.scale_log2, ubias));   // scale_log2 > 0: max commutes
        }
      }
      // move the reference maximum only when it grows a lot (or on the first finite value);
      // the decision is taken per warp so that the TMEM accesses stay convergent
      const bool grow = mx > m_ref + kRescaleThreshold;
      if (__any_sync(0xffffffffu, grow)) {
        if (j > 0) {
          const float alpha = grow ? exp2f(m_ref - mx) : 1.f;   // 0 when m_ref = -inf
          l *= alpha;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(lane_addr + C::kColO + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(lane_addr + C::kColO + c * 32, r);
          }
        }
        if (grow) m_ref = mx;
      }
      const float muse = m_ref == -INFINITY ? 0.f : m_ref;
      // pass 2: P = exp2(x - m), row sum, bf16 P over the first half of S's columns
#pragma unroll 1
      for (int c = 0; c < TK / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + C::kColS + c * 32, r);
        uint32_t p[16];
        if (table) {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float p0 = exp2f(fmaf(__uint_as_float(r[i]), a.scale_log2, s_kbias[j * TK + c * 32 + i] - muse));
            const float p1 = exp2f(fmaf(__uint_as_float(r[i + 1]), a.scale_log2, s_kbias[j * TK + c * 32 + i + 1] - muse));
            l += p0 + p1;
            p[i >> 1] = pack2(p0, p1);
          }
        } else if (dense_mask) {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const int col = j * TK + c * 32 + i;
            const float p0 = col <= climit ? exp2f(fmaf(__uint_as_float(r[i]), a.scale_log2, -muse)) : 0.f;
            const float p1 = col + 1 <= climit ? exp2f(fmaf(__uint_as_float(r[i + 1]), a.scale_log2, -muse)) : 0.f;
            l += p0 + p1;
            p[i >> 1] = pack2(p0, p1);
          }
        } else {
          const float off = ubias - muse;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float p0 = exp2f(fmaf(__uint_as_float(r[i]), a.scale_log2, off));
            const float p1 = exp2f(fmaf(__uint_as_float(r[i + 1]), a.scale_log2, off));
            l += p0 + p1;
            p[i >> 1] = pack2(p0, p1);
          }
        }
        tmem_st16(lane_addr + C::kColS + c * 16, p);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p);
    }
    // epilogue
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_o, 0, s_abort, status));
    if (ok) {
      tc_fence_after();
      const int qr = s_qrow[row];
      const float inv = 1.f / l;
      const float lse = (m_ref + log2f(l)) * 0.69314718055994531f;
      const size_t orow = t.orow_base + (size_t)(qr + t.odelta);
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + C::kColO + c * 32, r);
        if (qr >= 0) {
          if (t.partial || a.out_fp32) {
            float* dst = (t.partial ? a.part_o : reinterpret_cast<float*>(a.out)) + orow * D + c * 32;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv,
                                                                __uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.out) + orow * D + c * 32;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 v;
              v.x = pack2(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv);
              v.y = pack2(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
              v.z = pack2(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
              v.w = pack2(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
              *reinterpret_cast<uint4*>(dst + i) = v;
            }
          }
        }
      }
      if (qr >= 0) {
        if (t.partial) a.part_lse[orow] = lse;
        else a.lse[orow] = lse;
      }
    }
  } else if (warp == 4) {
    // =========================== MMA issue (one lane) ===========================================
    if (lane == 0) {
      constexpr uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
      constexpr uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
      bool ok = mbar_wait(bar_q, 0, s_abort, status);
      for (int j = 0; j < ntiles && ok; ++j) {
        const int s = j % C::NS;
        const uint32_t par = (j / C::NS) & 1;
        ok = mbar_wait(bar_kfull(s), par, s_abort, status);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t koff = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
          mma_ss(tmem + C::kColS, make_desc(ubase + C::kOffQ + koff, 16, 1024),
                 make_desc(ubase + C::kOffK + s * C::kTile + koff, 16, 1024), idesc_s, ks > 0);
        }
        umma_commit(bar_s);
        umma_commit(bar_kempty(s));
        ok = mbar_wait(bar_p, j & 1, s_abort, status);
        if (!ok) break;
        ok = mbar_wait(bar_vfull(s), par, s_abort, status);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk)
          mma_ts(tmem + C::kColO, tmem + C::kColS + kk * 8,
                 make_desc(ubase + C::kOffV + s * C::kTile + kk * 2048, 128 * 128, 1024), idesc_o, (j > 0 || kk > 0));
        umma_commit(bar_vempty(s));
        if (j == ntiles - 1) umma_commit(bar_o);
      }
    }
    __syncwarp();
  } else {
    // =========================== loaders: gather rows into swizzled tiles =======================
    const int lt = tid - 160;
    const __nv_bfloat16* qs = a.q + (size_t)t.seg * g.n * D;
    const __nv_bfloat16* ks = a.k + (size_t)t.seg * g.n * D;
    const __nv_bfloat16* vs = a.v + (size_t)t.seg * g.n * D;
    constexpr int CPR = D / 8;
    uint32_t pend[3] = {0u, 0u, 0u};
    int npend = 0;
    bool ok = true;
    auto retire_oldest = [&]() {
      cp_async_wait_le(npend - 1);
      fence_async_smem();
      mbar_arrive(pend[0]);
      pend[0] = pend[1]; pend[1] = pend[2];
      --npend;
    };
    auto gather = [&](uint32_t dst, const __nv_bfloat16* src, int kt, bool is_q, uint32_t full_bar) {
      for (int c = lt; c < 128 * CPR; c += kLoaderThreads) {
        const int row = c / CPR, cc = c % CPR;
        int gr;
        if (is_q) gr = s_qrow[row];
        else if (t.mode == 1) gr = s_kidx[kt * TK + row];
        else { const int i = kt * TK + row; gr = i < t.nk ? t.k0 + i : -1; }
        const uint32_t d = dst + tile_off(row, cc);
        if (gr >= 0) cp_async16(d, src + (size_t)gr * D + cc * 8);
        else st_shared_zero16(d);
      }
      cp_async_commit();
      pend[npend++] = full_bar;
      if (npend == 3) retire_oldest();
    };
    gather(ubase + C::kOffQ, qs, 0, true, bar_q);
    for (int j = 0; j < ntiles && ok; ++j) {
      const int s = j % C::NS;
      const int use = j / C::NS;
      if (use > 0) {
        while (npend) retire_oldest();
        ok = mbar_wait(bar_kempty(s), (use - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      gather(ubase + C::kOffK + s * C::kTile, ks, j, false, bar_kfull(s));
      if (use > 0) {
        while (npend) retire_oldest();
        ok = mbar_wait(bar_vempty(s), (use - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      gather(ubase + C::kOffV + s * C::kTile, vs, j, false, bar_vfull(s));
    }
    if (ok) { while (npend) retire_oldest(); }
    cp_async_wait_le(0);
  }

  // ---- teardown ------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
  }
}

}  // namespace

cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st) {
  if (a.total_tiles == 0) return cudaSuccess;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    kernel<<<a.total_tiles, 256, smem_bytes, st>>>(a, status);
    return cudaGetLastError();
  };
  if (a.g.d == 64) return go(attn_tc_kernel<64>, Cfg<64>::kTotal);
  return go(attn_tc_kernel<128>, Cfg<128>::kTotal);
}

}  // namespace hyperattn
