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
// One CTA per query tile of the forward schedule (same row tables, same sort and samples), key
// tiles of 128, all five products on the tcgen05 tensor cores with accumulators in TMEM (see
// bwd_tc_kernel); the three gradients are accumulated in fp32 with global reductions (a key
// tile is shared by every query tile that samples it, a query row by every level it appears in).
#include <cuda.h>
#include "attn_common.cuh"

namespace hyperattn {

bool encode_rows_map(CUtensorMap* m, const void* base, size_t rows, int d, int box_rows);   // attn_tc.cu

namespace {

// K and V as [G * n rows x d] bf16 tensors, 128-byte swizzle, box = 64 columns x 128 rows: key tiles of
// consecutive rows (causal leaves, unsorted nodes) arrive by TMA instead of through the load/store unit,
// which the reductions keep busy
struct alignas(64) BwdMaps {
  CUtensorMap k, v;
};


__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void st_shared_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
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

struct BwdArgs {
  AttnArgs a;
  const __nv_bfloat16* dout;   // [G, n, D]
  const float* lse;            // [G, n] final log-sum-exp of the forward pass (natural log)
  const float* delta;          // [G, n] <dO_i, O_i>
  float *dq, *dk, *dv;         // [G, n, D] fp32 accumulators, zeroed before the launch
  void* dq_final;              // dq_mode 1 / 2: dQ rows are written here directly (fp32 / bf16) instead of accumulated
  int dq_mode;                 // 0: a query row collects from several tiles (causal recursion): fp32 reductions into dq
  float scale;
  int table_keys;              // key columns of a node tile's row tables (block and samples, each padded to whole tiles)
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

// ---------------------------------------------------------------------------------------------
// One CTA per query tile, key tiles of 128, all five
// products on the 5th-generation tensor cores with operands in 128-byte-swizzled shared memory:
//     S  = Q K^T       A = Q  [query][d]   K-major,  B = K  [key][d]   K-major      -> TMEM cols   0..127
//     dP = dO V^T      A = dO [query][d]   K-major,  B = V  [key][d]   K-major      -> TMEM cols 128..255
//     dQ += dS K       A = dS [query][key] K-major,  B = K  [key][d]   MN-major     -> TMEM cols 256..256+d
//     dV  = P^T dO     A = P  [query][key] MN-major, B = dO [query][d]  MN-major     -> over S's columns
//     dK  = dS^T Q     A = dS [query][key] MN-major, B = Q  [query][d]  MN-major     -> over dP's columns
// 512 threads: threads t, t + 128, t + 256 and t + 384 share TMEM lane t mod 128 - query row t when P
// and dS are formed (each takes 32 of the tile's 128 key columns), key row t when dV and dK leave
// TMEM (the 2 d / 32 pieces of 32 columns are dealt round to the four groups of 128 threads).  Sixteen
// warps instead of eight hide a little more latency (2-3 % per call).  The phases of a key tile run one after the other (loads, S
// and dP, P and dS, the three gradient products, reductions): correct first, overlapped later.
constexpr int TKB = 128;   // keys per tile
constexpr unsigned long long kBwdWaitNs = 2000000000ull;

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// bounded wait: false after two seconds (the caller raises the status word and winds down)
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
    if (ok) return true;
    if ((it & 63u) == 63u) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kBwdWaitNs) return false;
    }
  }
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}\n"
               ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc) : "memory");
}
// packed fp32 pairs (two lanes per instruction)
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(__float_as_uint(lo)), "r"(__float_as_uint(hi)));
  return d;
}
__device__ __forceinline__ uint64_t pk2u(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a); hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
               "\ttcgen05.wait::ld.sync.aligned;\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr) : "memory");
}
// two loads in flight, one wait
__device__ __forceinline__ void tmem_ld32_pair(uint32_t ta, uint32_t (&a)[32], uint32_t tb, uint32_t (&b)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]), "=r"(a[6]), "=r"(a[7]),
                 "=r"(a[8]), "=r"(a[9]), "=r"(a[10]), "=r"(a[11]), "=r"(a[12]), "=r"(a[13]), "=r"(a[14]), "=r"(a[15]),
                 "=r"(a[16]), "=r"(a[17]), "=r"(a[18]), "=r"(a[19]), "=r"(a[20]), "=r"(a[21]), "=r"(a[22]), "=r"(a[23]),
                 "=r"(a[24]), "=r"(a[25]), "=r"(a[26]), "=r"(a[27]), "=r"(a[28]), "=r"(a[29]), "=r"(a[30]), "=r"(a[31])
               : "r"(ta) : "memory");
  tmem_ld32(tb, b);     // (its wait covers both loads)
#pragma unroll
  for (int i = 0; i < 32; ++i) asm volatile("" : "+r"(a[i]));    // no use of a[] may be scheduled above the wait
}

constexpr int kBwdThreads = 512;   // four threads per TMEM lane: 32 of a tile's 128 columns each

template <int D>
struct SmemTc {
  static constexpr int kQ = 128 * D * 2;              // Q, dO, K, V tiles: [128 rows x D]
  static constexpr int kP = 128 * TKB * 2;            // P, dS: [128 queries x 128 keys]
  static constexpr int kOffQ = 0, kOffdO = kQ, kOffK = 2 * kQ, kOffV = 3 * kQ, kOffP = 4 * kQ, kOffdS = 4 * kQ + kP;
  static constexpr int kOffMisc = 4 * kQ + 2 * kP;    // mbarrier, TMEM address, abort flag
  static constexpr int kOffRow = kOffMisc + 64;       // s_qrow [128]
  static constexpr int kFixed = kOffRow + 128 * 4;    // + 8 bytes per key column of the row tables
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1) bwd_tc_kernel(const __grid_constant__ BwdArgs b, const __grid_constant__ BwdMaps maps, int* status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using SM = SmemTc<D>;
  const AttnArgs& a = b.a;
  const Geometry& g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = tid & 127, part = tid >> 7;            // TMEM lane / tile row of this thread; which quarter of the work it takes
  const TileDesc t = decode_tile(a, blockIdx.x);
  if (t.nq <= 0) return;

  const uint32_t ubase = smem_u32(smem);
  const uint32_t uQ = ubase + SM::kOffQ, udO = ubase + SM::kOffdO, uK = ubase + SM::kOffK, uV = ubase + SM::kOffV;
  const uint32_t uP = ubase + SM::kOffP, udS = ubase + SM::kOffdS;
  const uint32_t bar = ubase + SM::kOffMisc;
  const uint32_t bar_kv = ubase + SM::kOffMisc + 8;       // K and V tile of consecutive rows landed (TMA)
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + SM::kOffMisc + 16);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + SM::kOffMisc + 32);
  int* s_qrow = reinterpret_cast<int*>(smem + SM::kOffRow);
  int* s_kidx = s_qrow + 128;                                    // [table_keys]
  float* s_kbias = reinterpret_cast<float*>(s_kidx + b.table_keys);

  const size_t seg_row0 = (size_t)t.seg * g.n;
  const __nv_bfloat16* qs = a.q + seg_row0 * D;
  const __nv_bfloat16* ks = a.k + seg_row0 * D;
  const __nv_bfloat16* vs = a.v + seg_row0 * D;
  const __nv_bfloat16* dos = b.dout + seg_row0 * D;

  // ---- row tables: key columns padded to whole tiles of 128 ----------------------------------
  int nkeys;
  if (t.mode == 1) {
    const int bpad = (g.b + TKB - 1) / TKB * TKB, mpad = (g.m + TKB - 1) / TKB * TKB;
    nkeys = bpad + mpad;
    const float wlog = g.m > 0 ? log2f((float)t.nk / (float)g.m) : 0.f;
    const int32_t* smp = a.samples + ((size_t)t.seg * g.nodes + t.node) * g.m;
    for (int i = tid; i < nkeys; i += kBwdThreads) {
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
    if (tid < 128) s_qrow[tid] = tid < t.nq ? t.qnode0 + a.perm_q[t.slice + t.spos0 + tid] : -1;
  } else {
    const int lim = t.causal ? min(t.nk, t.qk_off + t.nq) : t.nk;
    nkeys = (lim + TKB - 1) / TKB * TKB;
    if (tid < 128) s_qrow[tid] = tid < t.nq ? t.q0 + tid : -1;
  }
  if (tid == 0) {
    *s_abort = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_kv) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  constexpr int kTmemCols = 512;                       // S 128 | dP 128 | dQ D  (power of two)
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *s_tmem;
  const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  constexpr uint32_t colS = 0, colDP = 128, colDQ = 256;

  const int my_qrow = s_qrow[row];
  // (a padding row gets lse = +inf, so that all its weights are zero)
  const float lse2 = my_qrow >= 0 ? b.lse[seg_row0 + my_qrow] * 1.4426950408889634f : INFINITY;
  const float delta = my_qrow >= 0 ? b.delta[seg_row0 + my_qrow] : 0.f;

  auto krow_of = [&](int i) {          // segment-relative key row of key column i, -1: padding
    if (t.mode == 1) return s_kidx[i];
    return i < t.nk ? t.k0 + i : -1;
  };
  constexpr int CPR = D / 8;
  auto gather_rows = [&](uint32_t dst, const __nv_bfloat16* src, auto rowfn) {
#pragma unroll
    for (int i = 0; i < 128 * CPR / kBwdThreads; ++i) {
      const int c = tid + i * kBwdThreads;
      const int r = c / CPR, cc = c % CPR;
      const int gr = rowfn(r);
      const uint32_t d = dst + tile_off<128>(r, cc);
      if (gr >= 0) cp_async16(d, src + (size_t)gr * D + cc * 8);
      else st_shared_zero16(d);
    }
  };
  gather_rows(uQ, qs, [&](int r) { return s_qrow[r]; });
  gather_rows(udO, dos, [&](int r) { return s_qrow[r]; });

  // descriptors: low word = start >> 4 | (leading byte offset >> 4) << 16, high word = stride 1024 B | version | 128-byte swizzle
  constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  constexpr uint32_t kSlab = 128 * 128;                // bytes of one [128 rows x 64 columns] slab
  constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);
  constexpr uint32_t idesc_s = idesc_base | ((128u >> 3) << 17);                              // K-major x K-major, N = 128
  constexpr uint32_t idesc_dq = idesc_base | (1u << 16) | (((uint32_t)D >> 3) << 17);          // K-major x MN-major, N = D
  constexpr uint32_t idesc_t = idesc_base | (1u << 15) | (1u << 16) | (((uint32_t)D >> 3) << 17);   // MN-major x MN-major, N = D
  auto kmajor = [&](uint32_t base, int ks) { return ((base + (ks >> 2) * kSlab + (ks & 3) * 32) >> 4) | (1u << 16); };
  auto mnmajor = [&](uint32_t base, int kk) { return ((base + kk * 2048) >> 4) | ((kSlab >> 4) << 16); };

  // Rows leave TMEM one per thread, but a reduction instruction whose lanes hit 32 different rows costs
  // the L2 32 half-filled sectors: the warp's 32 rows x 32 columns pass through a 4 KB slice of shared
  // memory (the P tile's, idle at that point; chunks XOR-swizzled by row) and go out with eight lanes
  // per row, four rows per instruction.
  const uint32_t ustage = uP + warp * 4096;
  auto reduce_rows = [&](const uint32_t (&r)[32], float f, float* base, int grow, int c0, int store) {
    const int lane = tid & 31;
#pragma unroll
    for (int c = 0; c < 8; ++c)
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(ustage + lane * 128 + ((c ^ (lane & 7)) << 4)),
                   "f"(__uint_as_float(r[4 * c]) * f), "f"(__uint_as_float(r[4 * c + 1]) * f),
                   "f"(__uint_as_float(r[4 * c + 2]) * f), "f"(__uint_as_float(r[4 * c + 3]) * f) : "memory");
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int rr = 4 * it + (lane >> 3), c = lane & 7;
      const int gr = __shfl_sync(0xffffffffu, grow, rr);
      float4 v;
      asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                   : "r"(ustage + rr * 128 + ((c ^ (rr & 7)) << 4)) : "memory");
      if (gr >= 0) {
        const size_t el = (seg_row0 + gr) * D + c0 + 4 * c;
        if (store == 0) atomicAdd(reinterpret_cast<float4*>(base + el), v);
        else if (store == 1) *reinterpret_cast<float4*>(base + el) = v;
        else *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(base) + el) = make_uint2(pack2(v.x, v.y), pack2(v.z, v.w));
      }
    }
    __syncwarp();
  };
  const int ntiles = nkeys / TKB;
  uint32_t phase = 0;
  bool ok = true;
  const bool dense = t.mode != 1;
  auto load_kv = [&](int kt) {
    if (dense) {
      // consecutive rows: one TMA box per 64 columns (rows past the key range are masked, rows past the tensor are zeros)
      if (tid == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_kv), "r"((uint32_t)(2 * SM::kQ)) : "memory");
        const int y = (int)seg_row0 + t.k0 + kt * TKB;
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) {
          asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                       ::"r"(uK + sl * kSlab), "l"(&maps.k), "r"(sl * 64), "r"(y), "r"(bar_kv) : "memory");
          asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                       ::"r"(uV + sl * kSlab), "l"(&maps.v), "r"(sl * 64), "r"(y), "r"(bar_kv) : "memory");
        }
      }
    } else {
      gather_rows(uK, ks, [&](int r) { return krow_of(kt * TKB + r); });
      gather_rows(uV, vs, [&](int r) { return krow_of(kt * TKB + r); });
    }
    cp_async_commit();
  };
  if (ntiles > 0) load_kv(0);
  for (int kt = 0; kt < ntiles; ++kt) {
    // ---- this tile's K and V (requested while the previous tile's dV and dK left TMEM) ----------
    cp_async_wait<0>();
    if (dense && !mbar_wait_bounded(bar_kv, kt & 1)) *s_abort = 1;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    // ---- S = Q K^T, dP = dO V^T ----------------------------------------------------------------
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int s = 0; s < D / 16; ++s) mma_ss(tmem + colS, kmajor(uQ, s), kmajor(uK, s), desc_hi, idesc_s, s > 0);
#pragma unroll
      for (int s = 0; s < D / 16; ++s) mma_ss(tmem + colDP, kmajor(udO, s), kmajor(uV, s), desc_hi, idesc_s, s > 0);
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    }
    if (!mbar_wait_bounded(bar, phase)) *s_abort = 1;
    phase ^= 1;
    __syncthreads();
    if (*s_abort) { ok = false; break; }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // ---- P = C o exp(s - lse), dS = P (dP - delta): thread = query row ---------------------------
#pragma unroll 1
    for (int c0 = 32 * part; c0 < 32 * part + 32; c0 += 32) {
      uint32_t rs[32], rd[32];
      tmem_ld32_pair(lane_addr + colS + c0, rs, lane_addr + colDP + c0, rd);
      uint32_t pp[16], dd[16];
      const int colbase = kt * TKB + c0;
      // dense tiles need the mask only where the tile crosses the diagonal or the end of the keys
      const bool dense_mask = t.mode != 1 && (colbase + 32 > t.nk || (t.causal && colbase + 31 > t.qk_off));
      const uint64_t sc2 = pk2(a.scale_log2, a.scale_log2), nlse2 = pk2(-lse2, -lse2), ndel2 = pk2(-delta, -delta);
#pragma unroll
      for (int e = 0; e < 32; e += 4) {
        float4 bias = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t.mode == 1) bias = *reinterpret_cast<const float4*>(s_kbias + colbase + e);
        const uint64_t off2[2] = {t.mode == 1 ? fadd2(pk2(bias.x, bias.y), nlse2) : nlse2, t.mode == 1 ? fadd2(pk2(bias.z, bias.w), nlse2) : nlse2};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float x0, x1, p0, p1, d0, d1;
          upk2(ffma2(pk2u(rs[e + 2 * h], rs[e + 2 * h + 1]), sc2, off2[h]), x0, x1);
          if (dense_mask) {
            const int col = colbase + e + 2 * h;
            if (col >= t.nk || (t.causal && col > t.qk_off + row)) x0 = -INFINITY;
            if (col + 1 >= t.nk || (t.causal && col + 1 > t.qk_off + row)) x1 = -INFINITY;
          }
          asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p0) : "f"(x0));
          asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p1) : "f"(x1));
          upk2(fmul2(pk2(p0, p1), fadd2(pk2u(rd[e + 2 * h], rd[e + 2 * h + 1]), ndel2)), d0, d1);
          pp[(e >> 1) + h] = pack2(p0, p1);
          dd[(e >> 1) + h] = pack2(d0, d1);
        }
      }
      // row `tid`, key columns c0 .. c0+31 = 16-byte chunks c0/8 .. c0/8+3 of the [query][key] tiles
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const uint32_t off = tile_off<128>(row, c0 / 8 + q4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(uP + off), "r"(pp[4 * q4]), "r"(pp[4 * q4 + 1]), "r"(pp[4 * q4 + 2]), "r"(pp[4 * q4 + 3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(udS + off), "r"(dd[4 * q4]), "r"(dd[4 * q4 + 1]), "r"(dd[4 * q4 + 2]), "r"(dd[4 * q4 + 3]) : "memory");
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    // ---- dQ += dS K, dV = P^T dO, dK = dS^T Q -------------------------------------------------------
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int kk = 0; kk < TKB / 16; ++kk) mma_ss(tmem + colDQ, kmajor(udS, kk), mnmajor(uK, kk), desc_hi, idesc_dq, (kt > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
      for (int kk = 0; kk < 128 / 16; ++kk) mma_ss(tmem + colS, mnmajor(uP, kk), mnmajor(udO, kk), desc_hi, idesc_t, kk > 0);
#pragma unroll
      for (int kk = 0; kk < 128 / 16; ++kk) mma_ss(tmem + colDP, mnmajor(udS, kk), mnmajor(uQ, kk), desc_hi, idesc_t, kk > 0);
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    }
    if (!mbar_wait_bounded(bar, phase)) *s_abort = 1;
    phase ^= 1;
    __syncthreads();
    if (*s_abort) { ok = false; break; }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // ---- dV and dK of this key tile leave TMEM: thread = key row ----------------------------------
    {
      const int kr = krow_of(kt * TKB + row);
      // every product that read K and V has finished: the next tile's rows can come in meanwhile
      if (kt + 1 < ntiles) load_kv(kt + 1);
      // 2 * D / 32 pieces of 32 columns (dV first, then dK), every fourth one to each group of 128 threads
#pragma unroll 1
      for (int piece = part; piece < 2 * (D / 32); piece += 4) {
        const bool is_dk = piece >= D / 32;
        const int c0 = (piece % (D / 32)) * 32;
        uint32_t r[32];
        tmem_ld32(lane_addr + (is_dk ? colDP : colS) + c0, r);
        reduce_rows(r, is_dk ? b.scale : 1.f, is_dk ? b.dk : b.dv, kr, c0, 0);
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();   // S / dP columns and the K, V, P, dS tiles are free again
  }
  // ---- dQ: thread = query row (a row collects from every level it appears in) ---------------------
  if (ok && ntiles > 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
    for (int c0 = 32 * part; c0 < D; c0 += 128) {
      uint32_t r[32];
      tmem_ld32(lane_addr + colDQ + c0, r);
      // (without the causal recursion a query row belongs to exactly one tile: its dQ is final)
      reduce_rows(r, b.scale, b.dq_mode ? reinterpret_cast<float*>(b.dq_final) : b.dq, my_qrow, c0, b.dq_mode);
    }
  }
  if (!ok && tid == 0) atomicOr(status, 1 << 30);      // a bounded wait gave up
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
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
                            float* delta, float* dq, float* dk, float* dv, void* dq_final, int dq_mode, float scale, int* status, cudaStream_t st) {
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
  b.a = a; b.dout = d16; b.lse = lse; b.delta = delta; b.dq = dq; b.dk = dk; b.dv = dv; b.dq_final = dq_final; b.dq_mode = dq_mode; b.scale = scale;
  if (rows > 0x7fffffffull) return cudaErrorInvalidValue;            // TMA row coordinates are 32-bit
  BwdMaps maps;
  if (!encode_rows_map(&maps.k, a.k, rows, a.g.d, 128) || !encode_rows_map(&maps.v, a.v, rows, a.g.d, 128)) return cudaErrorInvalidValue;
  b.table_keys = a.g.sorted ? (a.g.b + TKB - 1) / TKB * TKB + (a.g.m + TKB - 1) / TKB * TKB : 0;
  if (b.table_keys > kMaxNodeKeys) return cudaErrorInvalidValue;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e2 = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes + kMaxNodeKeys * 8);
    if (e2 != cudaSuccess) return e2;
    kernel<<<a.total_tiles, kBwdThreads, smem_bytes + b.table_keys * 8, st>>>(b, maps, status);
    return cudaGetLastError();
  };
  if (a.g.d == 64) return go(bwd_tc_kernel<64>, SmemTc<64>::kFixed);
  return go(bwd_tc_kernel<128>, SmemTc<128>::kFixed);
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
