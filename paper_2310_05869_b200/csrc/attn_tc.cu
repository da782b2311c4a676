// Attention tiles on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 inputs.
//
// One CTA owns a PAIR of query tiles (2 x 128 rows) that are neighbours in the tile order of
// their leaf / recursion node, and walks once over the key tiles (128 keys each) that either
// of them needs:
//     S_i = Q_i K^T      tcgen05.mma, operands in 128B-swizzled shared memory, S_i in TMEM
//     P_i = exp2(S_i*c + bias - m)   softmax warpgroup i: one thread per query row (TMEM
//                                    lane); P_i is written back over S_i as bf16
//     O_i += P_i V       tcgen05.mma with P_i read from TMEM, V MN-major in shared memory
// which covers the block-diagonal part (Sec. 4), the sampled residual with weight N/m
// (Alg. 2 line 7) and the exact causal leaves (Sec. 3.1) in one loop.  The two query tiles
// of a 256-row block share every key tile, so K and V are fetched once for 256 rows, and
// while one warpgroup exponentiates, the tensor pipe works for the other one.  The running
// row maximum is only moved when it grows by more than 2^8 (the accumulators absorb the
// rest), so O is rarely rescaled; outputs are normalised by the sum of the bf16-rounded
// weights that the tensor cores actually used, the log-sum-exp by the unrounded sum.  Rows
// of Q, K, V are gathered from their original places through the sortLSH permutations by
// three loader warps with 16-byte cp.async copies; nothing permuted is ever written to HBM.
//
// Warp roles (384 threads): warps 0-3 and 4-7 softmax + epilogue of query tile 0 and 1,
// warp 8 MMA issue + TMEM allocation (all 512 columns: S0 S1 O0 O1), warps 9-11 loaders.
// Every mbarrier wait is bounded: on a timeout the CTA raises the device status word,
// drains its copies, frees its TMEM and returns.
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
  static constexpr int NS = (D == 64) ? 4 : 2;        // K stages and V stages
  static constexpr int kTile = 128 * D * 2;           // bytes of one 128-row tile
  static constexpr int kOffQ = 0;                     // Q0, Q1
  static constexpr int kOffK = 2 * kTile;
  static constexpr int kOffV = kOffK + NS * kTile;
  static constexpr int kOffIdx = kOffV + NS * kTile;              // int [kMaxNodeKeys] key rows
  static constexpr int kOffMask = kOffIdx + kMaxNodeKeys * 4;     // uint32 [2][kMaxNodeKeys/32] masked-column bits
  static constexpr int kOffQrow = kOffMask + 2 * (kMaxNodeKeys / 32) * 4;   // int [2][128]
  static constexpr int kOffBar = kOffQrow + 2 * 128 * 4;
  static constexpr int kNumBar = 7 + 4 * NS;
  static constexpr int kOffMisc = kOffBar + 8 * kNumBar;          // tmem slot, abort flag
  static constexpr int kTotal = kOffMisc + 16;
  static constexpr int kTmemCols = 512;
  static constexpr int kColS = 0;                     // S_i at kColS + 128 i
  static constexpr int kColO = 256;                   // O_i at kColO + D i
};

// One query tile of the pair.
struct QTile {
  int valid;
  int nq;        // valid rows
  int q0;        // dense: first query row (segment-relative)
  int tt;        // dense causal: index of the diagonal key tile
  int beta;      // node: block
  int spos0;     // node: first sorted position
};

struct PairDesc {
  int mode;            // 0 dense, 1 node
  int seg;
  QTile qt[2];
  int causal;          // dense
  int k0, nk;          // dense: key range; node: first key row of the node and N
  int qnode0;          // node: first query row of the node
  size_t slice;        // node: slice offset in perm_q / perm_k / rank_k
  int node;            // node: heap index
  int nbA, nbB, nsmp;  // node: key tiles of block A, of block B (0 if shared), of the samples
  int ntiles;          // key tiles walked
  size_t orow_base; int odelta; int partial;
};

__device__ __forceinline__ PairDesc decode_pair(const AttnArgs& a, int pair) {
  const Geometry& g = a.g;
  PairDesc t;
  t.partial = !a.direct;
  t.qt[0].valid = 1; t.qt[1].valid = 0;
  t.nbA = t.nbB = t.nsmp = 0;
  int s, q0n, k0n;
  if (pair < a.n_leaf_pairs) {
    const int per = g.G * a.leaves_per_seg;
    const int uu = a.pairs_per_leaf - 1 - pair / per;       // heavy pairs first
    const int rem = pair % per;
    t.seg = rem / a.leaves_per_seg;
    const int leaf = rem % a.leaves_per_seg;
    t.mode = 0; t.causal = a.dense_causal;
    t.k0 = leaf * g.leaf; t.nk = g.leaf;
    for (int i = 0; i < 2; ++i) {
      const int tt = 2 * uu + i;
      t.qt[i].valid = tt < a.tiles_per_leaf;
      t.qt[i].tt = tt;
      t.qt[i].q0 = t.k0 + tt * kTileQ;
      t.qt[i].nq = min(kTileQ, g.leaf - tt * kTileQ);
    }
    t.orow_base = (size_t)t.seg * g.n; t.odelta = 0;
  } else {
    int level = 0;
    while (level + 1 < g.levels && pair >= a.level_pair_start[level + 1]) ++level;
    int idx = pair - a.level_pair_start[level];
    node_rows(g, level, 0, s, q0n, k0n);
    const int nodes_lvl = g.causal ? (1 << level) : 1;
    const int sorted = a.level_sorted[level];
    const int tiles_node = sorted ? (s / g.b) * a.tiles_per_block : (s + kTileQ - 1) / kTileQ;
    const int pairs_node = (tiles_node + 1) / 2;
    const int pn = idx % pairs_node; idx /= pairs_node;
    const int j = idx % nodes_lvl;
    t.seg = idx / nodes_lvl;
    node_rows(g, level, j, s, q0n, k0n);
    t.k0 = k0n; t.nk = s; t.qnode0 = q0n; t.causal = 0;
    for (int i = 0; i < 2; ++i) {
      const int tn = 2 * pn + i;
      QTile& q = t.qt[i];
      q.valid = tn < tiles_node;
      q.tt = 0;
      if (sorted) {
        q.beta = tn / a.tiles_per_block;
        const int sub = tn % a.tiles_per_block;
        q.spos0 = q.beta * g.b + sub * kTileQ;
        q.nq = min(kTileQ, g.b - sub * kTileQ);
        q.q0 = 0;
      } else {
        q.q0 = q0n + tn * kTileQ;
        q.nq = min(kTileQ, s - tn * kTileQ);
      }
    }
    t.mode = sorted;
    if (sorted) {
      t.slice = ((size_t)level * g.G + t.seg) * g.nl + (g.causal ? (size_t)j * s : 0);
      t.node = g.causal ? (1 << level) - 1 + j : 0;
      const int bt = (g.b + TK - 1) / TK;
      t.nbA = bt;
      t.nbB = (t.qt[1].valid && t.qt[1].beta != t.qt[0].beta) ? bt : 0;
      t.nsmp = (g.m + TK - 1) / TK;
    }
    if (a.direct) { t.orow_base = (size_t)t.seg * g.n; t.odelta = 0; }
    else { t.orow_base = (size_t)g.G * g.n + (size_t)level * g.G * g.nl + (size_t)t.seg * g.nl + (size_t)j * s; t.odelta = -q0n; }
  }
  if (t.mode == 1) {
    t.ntiles = t.nbA + t.nbB + t.nsmp;
  } else {
    const QTile& last = t.qt[1].valid ? t.qt[1] : t.qt[0];
    const int lim = t.causal ? min(t.nk, last.tt * kTileQ + last.nq) : t.nk;
    t.ntiles = (lim + TK - 1) / TK;
  }
  return t;
}

// does query tile i of the pair look at key tile j ?
__device__ __forceinline__ bool tile_active(const PairDesc& t, int i, int j) {
  if (!t.qt[i].valid) return false;
  if (t.mode == 0) return !t.causal || j <= t.qt[i].tt;
  if (j >= t.nbA + t.nbB) return true;                         // samples: both
  if (j < t.nbA) return i == 0 || t.nbB == 0;                  // block of tile 0 (shared when nbB == 0)
  return i == 1;                                               // block of tile 1
}

template <int D>
__global__ void __launch_bounds__(384, 1) attn_tc_kernel(const __grid_constant__ AttnArgs a, int* status) {
  using C = Cfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  int* s_kidx = reinterpret_cast<int*>(smem + C::kOffIdx);
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem + C::kOffMask);     // [2][kMaxNodeKeys/32]
  int* s_qrow = reinterpret_cast<int*>(smem + C::kOffQrow);               // [2][128]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);
  constexpr int MW = kMaxNodeKeys / 32;

  const uint32_t ubase = smem_u32(smem);
  const uint32_t bar0 = ubase + C::kOffBar;
  const uint32_t bar_q = bar0;
  auto bar_s = [&](int i) { return bar0 + 8 + 8 * i; };
  auto bar_p = [&](int i) { return bar0 + 24 + 8 * i; };
  auto bar_o = [&](int i) { return bar0 + 40 + 8 * i; };
  auto bar_kfull = [&](int s) { return bar0 + 56 + 8 * s; };
  auto bar_kempty = [&](int s) { return bar0 + 56 + 8 * (C::NS + s); };
  auto bar_vfull = [&](int s) { return bar0 + 56 + 8 * (2 * C::NS + s); };
  auto bar_vempty = [&](int s) { return bar0 + 56 + 8 * (3 * C::NS + s); };

  const Geometry& g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const PairDesc t = decode_pair(a, blockIdx.x);

  // A CTA of a launch in which some wait already timed out returns at once (nothing allocated
  // yet), so a stuck launch drains quickly instead of timing out tile after tile.
  if (tid == 0) *s_abort = *reinterpret_cast<volatile int*>(status);
  __syncthreads();
  if (*s_abort) return;
  __syncthreads();

  // ---- setup: barriers, TMEM, row tables ----------------------------------------------------
  if (tid == 0) {
    mbar_init(bar_q, kLoaderThreads);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_s(i), 1); mbar_init(bar_p(i), 128); mbar_init(bar_o(i), 1); }
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(bar_kfull(s), kLoaderThreads);
      mbar_init(bar_vfull(s), kLoaderThreads);
      mbar_init(bar_kempty(s), 1);
      mbar_init(bar_vempty(s), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < 2 * MW; i += 384) s_mask[i] = 0;
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  __syncthreads();

  float wlog = 0.f;  // log2(N/m): weight of a sampled column
  if (t.mode == 1) {
    const int bpad = t.nbA * TK;
    const int ncols = t.ntiles * TK;
    wlog = g.m > 0 ? log2f((float)t.nk / (float)g.m) : 0.f;
    const int32_t* smp = a.samples + ((size_t)t.seg * g.nodes + t.node) * g.m;
    for (int i = tid; i < ncols; i += 384) {
      int idx = -1;
      bool masked[2] = {true, true};
      if (i < (t.nbA + t.nbB) * TK) {
        const int which = i >= bpad;                  // 0: block of tile 0, 1: block of tile 1
        const int c = i - which * bpad;
        if (c < g.b) {
          idx = t.k0 + a.perm_k[t.slice + (size_t)t.qt[which].beta * g.b + c];
          masked[0] = masked[1] = false;
        }
      } else {
        const int c = i - (t.nbA + t.nbB) * TK;
        if (c < g.m) {
          const int l = smp[c];
          idx = t.k0 + l;
          const int blk = a.rank_k[t.slice + l] / g.b;
          masked[0] = blk == t.qt[0].beta;            // the factor (1 - M^H) of Alg. 2 line 7
          masked[1] = t.qt[1].valid && blk == t.qt[1].beta;
        }
      }
      s_kidx[i] = idx;
      if (masked[0]) atomicOr(&s_mask[i >> 5], 1u << (i & 31));
      if (masked[1]) atomicOr(&s_mask[MW + (i >> 5)], 1u << (i & 31));
    }
    if (tid < 2 * kTileQ) {
      const int i = tid >> 7, r = tid & 127;
      const QTile& q = t.qt[i];
      s_qrow[tid] = (q.valid && r < q.nq) ? t.qnode0 + a.perm_q[t.slice + q.spos0 + r] : -1;
    }
  } else {
    if (tid < 2 * kTileQ) {
      const int i = tid >> 7, r = tid & 127;
      const QTile& q = t.qt[i];
      s_qrow[tid] = (q.valid && r < q.nq) ? q.q0 + r : -1;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const int ntiles = t.ntiles;

  if (warp < 8) {
    // ================= softmax + epilogue of query tile i: thread = query row ==================
    const int i = warp >> 2;
    const int row = tid & 127;
    const QTile& q = t.qt[i];
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t colS = C::kColS + 128 * i, colO = C::kColO + D * i;
    float m_ref = -INFINITY, l = 0.f, lr = 0.f;     // l: unrounded row sum, lr: sum of the bf16 weights
    bool ok = true;
    int na = 0;                                     // active tiles seen
    for (int j = 0; j < ntiles && ok; ++j) {
      if (!tile_active(t, i, j)) continue;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s(i), na & 1, s_abort, status));   // warp-uniform: TMEM ops are .aligned
      if (!ok) break;
      tc_fence_after();
      // mask kind of this (query tile, key tile): uniform over the warpgroup
      bool table = false, dense_mask = false;
      float ubias = 0.f;
      int climit = 0;                               // dense: last visible column of this row
      if (t.mode == 1) {
        const uint32_t* mw = s_mask + i * MW + j * (TK / 32);
        table = (mw[0] | mw[1] | mw[2] | mw[3]) != 0;
        ubias = (j < t.nbA + t.nbB) ? 0.f : wlog;
      } else {
        dense_mask = (j * TK + TK > t.nk) || (t.causal && j == q.tt);
        climit = t.causal ? min(t.nk - 1, q.tt * kTileQ + row) : t.nk - 1;
      }
      // pass 1: row maximum of the tile
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < TK / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + colS + c * 32, r);
        if (table) {
          const uint32_t bits = s_mask[i * MW + j * (TK / 32) + c];
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (!((bits >> e) & 1u)) mx = fmaxf(mx, __uint_as_float(r[e]));
        } else if (dense_mask) {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (j * TK + c * 32 + e <= climit) mx = fmaxf(mx, __uint_as_float(r[e]));
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
        }
      }
      mx = fmaf(mx, a.scale_log2, ubias);           // scale_log2 > 0: the maximum commutes with it
      // move the reference maximum only when it grows a lot (or on the first finite value);
      // the decision is taken per warp so that the TMEM accesses stay convergent
      const bool grow = mx > m_ref + kRescaleThreshold;
      if (__any_sync(0xffffffffu, grow)) {
        if (na > 0) {
          const float alpha = grow ? exp2f(m_ref - mx) : 1.f;   // 0 when m_ref = -inf
          l *= alpha; lr *= alpha;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(lane_addr + colO + c * 32, r);
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st32(lane_addr + colO + c * 32, r);
          }
        }
        if (grow) m_ref = mx;
      }
      const float off = ubias - (m_ref == -INFINITY ? 0.f : m_ref);
      // pass 2: P = exp2(x - m), row sums, bf16 P over the first half of S's columns
#pragma unroll 1
      for (int c = 0; c < TK / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + colS + c * 32, r);
        uint32_t p[16];
        uint32_t vis = 0xffffffffu;                 // visible columns of this chunk
        if (table) vis = ~s_mask[i * MW + j * (TK / 32) + c];
        else if (dense_mask) {
          const int rel = climit - (j * TK + c * 32);           // columns 0..rel visible
          vis = rel >= 31 ? 0xffffffffu : (rel < 0 ? 0u : ((2u << rel) - 1u));
        }
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float p0 = exp2f(fmaf(__uint_as_float(r[e]), a.scale_log2, off));
          float p1 = exp2f(fmaf(__uint_as_float(r[e + 1]), a.scale_log2, off));
          if (table || dense_mask) {
            if (!((vis >> e) & 1u)) p0 = 0.f;
            if (!((vis >> (e + 1)) & 1u)) p1 = 0.f;
          }
          l += p0 + p1;
          const uint32_t w = pack2(p0, p1);
          lr += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
          p[e >> 1] = w;
        }
        tmem_st16(lane_addr + colS + c * 16, p);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p(i));
      ++na;
    }
    // epilogue
    if (q.valid) {
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_o(i), 0, s_abort, status));
      if (ok) {
        tc_fence_after();
        const int qr = s_qrow[i * 128 + row];
        const float inv = 1.f / lr;
        const float lse = (m_ref + log2f(l)) * 0.69314718055994531f;
        const size_t orow = t.orow_base + (size_t)(qr + t.odelta);
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(lane_addr + colO + c * 32, r);
          if (qr >= 0) {
            if (t.partial || a.out_fp32) {
              float* dst = (t.partial ? a.part_o : reinterpret_cast<float*>(a.out)) + orow * D + c * 32;
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4*>(dst + e) = make_float4(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv,
                                                                  __uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            } else {
              __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.out) + orow * D + c * 32;
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint4 v;
                v.x = pack2(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
                v.y = pack2(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
                v.z = pack2(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
                v.w = pack2(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
                *reinterpret_cast<uint4*>(dst + e) = v;
              }
            }
          }
        }
        if (qr >= 0) {
          if (t.partial) a.part_lse[orow] = lse;
          else a.lse[orow] = lse;
        }
      }
    }
  } else if (warp == 8) {
    // ================= MMA issue (one lane) ===========================================================
    if (lane == 0) {
      constexpr uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
      constexpr uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
      bool ok = mbar_wait(bar_q, 0, s_abort, status);
      int done[2] = {0, 0};        // PV steps issued per query tile
      int pend[2] = {-1, -1};      // key tile whose P_i is awaited
      int total[2] = {0, 0};
      for (int j = 0; j < ntiles; ++j) { total[0] += tile_active(t, 0, j); total[1] += tile_active(t, 1, j); }
      // PV_i of the pending key tile: needs P_i (softmax) and V of that tile
      auto flush_pv = [&](int i) {
        const int jp = pend[i];
        const int s = jp % C::NS;
        ok = mbar_wait(bar_p(i), done[i] & 1, s_abort, status);
        if (!ok) return;
        ok = mbar_wait(bar_vfull(s), (jp / C::NS) & 1, s_abort, status);
        if (!ok) return;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk)
          mma_ts(tmem + C::kColO + D * i, tmem + C::kColS + 128 * i + kk * 8,
                 make_desc(ubase + C::kOffV + s * C::kTile + kk * 2048, 128 * 128, 1024), idesc_o, (done[i] > 0 || kk > 0));
        ++done[i];
        pend[i] = -1;
        // V of tile jp is free once every query tile that uses it has issued its PV
        const int other = 1 - i;
        if (!tile_active(t, other, jp) || pend[other] != jp) umma_commit(bar_vempty(s));
        if (done[i] == total[i]) umma_commit(bar_o(i));
      };
      for (int j = 0; j < ntiles && ok; ++j) {
        const int s = j % C::NS;
        bool waited_k = false;
        for (int i = 0; i < 2 && ok; ++i) {
          if (pend[i] >= 0) flush_pv(i);
          if (!ok) break;
          if (!tile_active(t, i, j)) continue;
          if (!waited_k) {
            ok = mbar_wait(bar_kfull(s), (j / C::NS) & 1, s_abort, status);
            if (!ok) break;
            tc_fence_after();
            waited_k = true;
          }
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t koff = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
            mma_ss(tmem + C::kColS + 128 * i, make_desc(ubase + C::kOffQ + i * C::kTile + koff, 16, 1024),
                   make_desc(ubase + C::kOffK + s * C::kTile + koff, 16, 1024), idesc_s, ks > 0);
          }
          umma_commit(bar_s(i));
          pend[i] = j;
          // K of tile j is free once the last query tile that uses it has issued its S
          if (i == 1 || !tile_active(t, 1, j)) umma_commit(bar_kempty(s));
        }
      }
      for (int i = 0; i < 2 && ok; ++i)
        if (pend[i] >= 0) flush_pv(i);
    }
    __syncwarp();
  } else {
    // ================= loaders: gather rows into swizzled tiles ======================================
    const int lt = tid - 288;
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
    // kind 0/1: query tile 0/1 (both under one barrier), 2: key tile kt
    auto gather_rows = [&](uint32_t dst, const __nv_bfloat16* src, int kind, int kt) {
      for (int c = lt; c < 128 * CPR; c += kLoaderThreads) {
        const int row = c / CPR, cc = c % CPR;
        int gr;
        if (kind < 2) gr = s_qrow[kind * 128 + row];
        else if (t.mode == 1) gr = s_kidx[kt * TK + row];
        else { const int i = kt * TK + row; gr = i < t.nk ? t.k0 + i : -1; }
        const uint32_t d = dst + tile_off(row, cc);
        if (gr >= 0) cp_async16(d, src + (size_t)gr * D + cc * 8);
        else st_shared_zero16(d);
      }
    };
    auto committed = [&](uint32_t full_bar) {
      cp_async_commit();
      pend[npend++] = full_bar;
      if (npend == 3) retire_oldest();
    };
    gather_rows(ubase + C::kOffQ, qs, 0, 0);
    gather_rows(ubase + C::kOffQ + C::kTile, qs, 1, 0);
    committed(bar_q);
    for (int j = 0; j < ntiles && ok; ++j) {
      const int s = j % C::NS;
      const int use = j / C::NS;
      if (use > 0) {
        while (npend) retire_oldest();
        ok = mbar_wait(bar_kempty(s), (use - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      gather_rows(ubase + C::kOffK + s * C::kTile, ks, 2, j);
      committed(bar_kfull(s));
      if (use > 0) {
        while (npend) retire_oldest();
        ok = mbar_wait(bar_vempty(s), (use - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      gather_rows(ubase + C::kOffV + s * C::kTile, vs, 2, j);
      committed(bar_vfull(s));
    }
    if (ok) { while (npend) retire_oldest(); }
    cp_async_wait_le(0);
  }

  // ---- teardown ------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
  }
}

}  // namespace

cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st) {
  if (a.total_pairs == 0) return cudaSuccess;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    kernel<<<a.total_pairs, 384, smem_bytes, st>>>(a, status);
    return cudaGetLastError();
  };
  if (a.g.d == 64) return go(attn_tc_kernel<64>, Cfg<64>::kTotal);
  return go(attn_tc_kernel<128>, Cfg<128>::kTotal);
}

}  // namespace hyperattn
