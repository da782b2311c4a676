// Attention tiles on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 inputs.
//
// One CTA owns a PAIR of query tiles (2 x 128 rows) that are neighbours in the tile order of
// their leaf / recursion node, and walks once over the key tiles (64 keys each) that either
// of them needs:
//     S_i = Q_i K^T      tcgen05.mma, operands in 128B-swizzled shared memory, S_i in TMEM
//     P_i = exp2(S_i*c + bias - m)   softmax warpgroup i: one thread per query row (TMEM
//                                    lane); P_i is written back over S_i as bf16
//     O_i += P_i V       tcgen05.mma with P_i read from TMEM, V MN-major in shared memory
// which covers the block-diagonal part (Sec. 4), the sampled residual with weight N/m
// (Alg. 2 line 7) and the exact causal leaves (Sec. 3.1) in one loop.  The two query tiles
// of a 256-row block share every key tile, so K and V are fetched once for 256 rows, and
// every warpgroup has two S buffers in TMEM, so the tensor pipe computes the scores of the next
// key tile while the warpgroup exponentiates the current one.  The running
// row maximum is only moved when it grows by more than 2^32 (the accumulators absorb the
// rest), so O is rarely rescaled; outputs are normalised by the sum of the bf16-rounded
// weights that the tensor cores actually used (d = 64: accumulated by the tensor cores
// themselves, in an extra column of O whose B operand is a slab of ones; d = 128: in
// registers), the log-sum-exp by the unrounded sum.  Rows
// of Q, K, V come from their original places: tiles of consecutive rows (causal leaves) as
// one TMA box per 64 columns, tiles of sorted or sampled rows gathered through the sortLSH
// permutations with 16-byte cp.async copies into the same 128B-swizzled operand layout;
// nothing permuted is ever written to HBM.  (The TMA row gather, tile::gather4, was measured
// at about 100 cycles of issue per four rows and warp: too slow for this.)
//
// Warp roles (384 threads): warps 0-3 and 4-7 softmax + epilogue of query tile 0 and 1,
// warps 8 and 9 MMA issue for query tile 0 and 1 (warp 8 also allocates TMEM, all 512
// columns: per query tile two S buffers of 64, then O0, O1), warp 10 prepares work items (row tables of the
// NEXT item while this one computes, TMA boxes of Q), warp 11 streams K / V tiles through
// the stage ring, across item boundaries.  Gathered Q tiles are fetched by the 256 softmax
// threads, for the next item, right before they write the current item's results.
// Every mbarrier wait is bounded: on a timeout the CTA raises the device status word,
// drains its copies, frees its TMEM and returns.
#include <cstdlib>
#include <cuda.h>
#include "attn_common.cuh"

namespace hyperattn {
namespace {

// tensor maps of Q, K, V as [G * n rows x d] bf16 tensors, 128-byte swizzle; box = 64 columns x
// 128 rows (Q) or 64 rows (K, V): one slab of an operand tile
struct alignas(64) TmaMaps {
  CUtensorMap q, k, v;
};

constexpr int TK = 64;                  // keys per tile
#ifndef HA_WAIT_LIMIT_NS
#define HA_WAIT_LIMIT_NS 2000000000ull
#endif
constexpr unsigned long long kWaitLimitNs = HA_WAIT_LIMIT_NS;   // every mbarrier wait gives up after 2 s
// Test build only (-DHA_TEST_DROP_ARRIVAL, never in the shipped library): when armed, the K / V streamer of one CTA
// leaves out the copies of one V tile once, so that the wait for that tile runs out and the give-up path can be
// exercised without any fault.
#ifdef HA_TEST_DROP_ARRIVAL
__device__ int g_test_drop_armed;
#endif
constexpr float kRescaleThreshold = 32.f;   // octaves the scores may exceed the reference before it moves
constexpr float kTileSumLimit = 1099511627776.f;   // 2^40: a tile whose weights sum to more has a score > 2^34 above the reference

// Optional per-role cycle counters (compile with -DHA_TC_TIMING; never in the shipped build).
#ifdef HA_TC_TIMING
__device__ unsigned long long g_tc_timing[48];
#define HA_T0(var) const long long var = clock64()
#define HA_TACC(slot, var) atomicAdd(&g_tc_timing[slot], (unsigned long long)(clock64() - var))
#define HA_LDECL(name) long long name = 0
#define HA_LACC(name, var) name += clock64() - var
#define HA_LFLUSH(slot, name) atomicAdd(&g_tc_timing[slot], (unsigned long long)(name))
#else
#define HA_T0(var)
#define HA_TACC(slot, var)
#define HA_LDECL(name)
#define HA_LACC(name, var)
#define HA_LFLUSH(slot, name)
#endif

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ---------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One potentially-blocking probe: the hardware may park the warp for up to the hinted time (ns)
// and wakes it when the phase completes, so waiting warps leave the issue slots to the others.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
               : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
  return ok != 0;
}
// returns false when the wait gave up (timeout or another thread aborted)
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// SLEEP_NS: back-off between probes, so that waiting warps do not take issue slots from the
// warps that compute (every role waits far more often than it works)
template <int SLEEP_NS = 32, int SITE = 1>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    if (mbar_try(bar, parity)) return true;
    __nanosleep(SLEEP_NS);
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  atomicOr(status, 1 << SITE);     // bit mask of the wait sites that gave up
  return false;
}

// the slow path of a wait, out of line; SITE tags the wait in the status word
template <int SITE>
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  return mbar_wait<20, SITE>(bar, parity, abort_flag, status);
}
// one probe inline (the common case for the MMA issuers: what they wait for is usually there)
template <int SITE>
__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow<SITE>(bar, parity, abort_flag, status);
}

// ---- tcgen05 ----------------------------------------------------------------------------
// tcgen05.mma with shared-memory descriptors given as (low, high) 32-bit words: only the low word ever changes
// (low word = start address >> 4 | (leading byte offset >> 4) << 16, high word = stride byte offset >> 4 |
// descriptor version 1 << 14 | 128-byte swizzle 2 << 29); [a_tmem]: the A operand read from TMEM
__device__ __forceinline__ void mma_ss2(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}\n"
               ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts2(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}\n"
               ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// issue without waiting; the data is valid only after tmem_ld32_wait on the same registers
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
}
// waits for every outstanding TMEM load of this thread; the registers are listed as
// read-write operands so that no use of them can be scheduled above the wait
__device__ __forceinline__ void tmem_ld32_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16_wait(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :: "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
#ifdef HA_EXP_FAKE
  asm("mul.f32 %0, %1, 0f00000000;" : "=f"(y) : "f"(x));     // timing experiment only: results are meaningless
#else
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
#endif
  return y;
}
// packed pairs of fp32 (one instruction, two lanes)
__device__ __forceinline__ uint64_t pack_u2(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) { return pack_u2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi) {
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

// ---- copies -----------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
// the executing thread's arrival on the mbarrier happens when all its earlier cp.async have landed
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// One TMA box (64 columns x the map's box rows, starting at column x, row y) into a
// 128B-swizzled slab; completion is counted in bytes on the mbarrier.
__device__ __forceinline__ void tma_tile(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// announces bytes to the current phase without arriving
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Teardown only: waits (bounded, whatever the abort flag says) until a phase that this warp
// armed has received all its bytes, so that no copy is in flight into the CTA's shared
// memory when it exits.
__device__ __noinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = global_ns();
  for (unsigned it = 0;; ++it) {
    if (mbar_try(bar, parity)) return;
    if ((it & 15u) == 15u && global_ns() - t0 > kWaitLimitNs) return;
  }
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// byte offset of 16-byte chunk c of row `row` in a [ROWS x D] bf16 tile: D/64 slabs of
// [ROWS rows x 128 B], 128-byte swizzle inside each slab (the canonical tcgen05 layout)
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int row, int c) {
  return (uint32_t)((c >> 3) * (ROWS * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4));
}

// Tiles with masked columns (a minority: the diagonal tiles of a causal leaf, padding, sampled
// columns that fall into the query tile's own block): the masked scores are overwritten with
// -inf in TMEM before the tile is read, so that the hot loop carries no mask code at all.
// vis: one bit per column, 1 = visible.  All 32 lanes call it together.
__device__ __noinline__ void mask_scores(uint32_t sbase, uint32_t visa, uint32_t visb) {
  uint32_t r[16];
#pragma unroll 1
  for (int gcol = 0; gcol < 4; ++gcol) {
    const uint32_t vis16 = ((gcol < 2 ? visa : visb) >> (16 * (gcol & 1))) & 0xffffu;
    if (__all_sync(0xffffffffu, vis16 == 0xffffu)) continue;      // warp-uniform: TMEM accesses stay convergent
    tmem_ld16_issue(sbase + 16 * gcol, r);
    tmem_ld16_wait(r);
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if (!((vis16 >> e) & 1u)) r[e] = 0xff800000u;
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
                 ::"r"(sbase + 16 * gcol), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
  }
  tmem_wait_st();
}

// Rare path of the online softmax: multiply the O columns a row has accumulated so far by
// alpha (a power of two, so nothing is re-rounded).  Kept out of line: the hot loop should
// stay small.  All 32 lanes call it together (TMEM accesses are warp-wide).
__device__ __noinline__ void rescale_row(uint32_t o_addr, int ocols, float alpha) {
  uint32_t r[16];
  for (int c = 0; c < ocols; c += 16) {
    tmem_ld16_issue(o_addr + c, r);
    tmem_ld16_wait(r);
#pragma unroll
    for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
                 ::"r"(o_addr + c), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
  }
  tmem_wait_st();
}

// One query tile of the pair.  The key tiles it looks at are two runs of the pair's tile
// list: [s1, s1 + n1) and [s2, s2 + n2).
struct QTile {
  int valid;
  int nq;        // valid rows
  int q0;        // dense: first query row (segment-relative)
  int row0;      // dense causal: local index of the tile's first row (relative to the first key)
  int beta;      // node: block
  int spos0;     // node: first sorted position
  int s1, n1, s2, n2;
};

struct PairDesc {
  int mode;            // 0 dense, 1 node
  int seg;
  int causal;          // dense
  int k0, nk;          // dense: key range; node: first key row of the node and N
  int qnode0;          // node: first query row of the node
  size_t slice;        // node: slice offset in perm_q / perm_k / rank_k
  int node;            // node: heap index
  int nq_node, bq;     // node: query rows of the node, rows per group of sorted queries
  int nbA, nbB, nsmp;  // node: key tiles of block A, of block B (0 if shared), of the samples
  float bias_max;      // node, weighted sampling: the largest log2 weight among the samples
  int ntiles;          // key tiles walked
  size_t orow_base; int odelta; int partial;
};

// what every role needs to know about a work item; decoded once, by the item preparer
struct ItemDesc {
  PairDesc t;
  QTile qa, qb;
};

template <int D>
struct Cfg {
  static constexpr int NS = (D == 64) ? 8 : 4;        // K stages and V stages
  static constexpr int kQTile = 128 * D * 2;          // bytes of one 128-row query tile
  static constexpr int kTile = TK * D * 2;            // bytes of one key / value tile
  static constexpr int kOffQ = 0;                     // Q0, Q1
  static constexpr int kOffK = 2 * kQTile;
  static constexpr int kOffV = kOffK + NS * kTile;
  // row tables, two sets (the loaders build the set of the next work item while this one runs)
  static constexpr int kOffIdx = kOffV + NS * kTile;              // int [2][kMaxNodeKeys] key rows
  static constexpr int kOffMask = kOffIdx + 2 * kMaxNodeKeys * 4; // uint32 [2][2][kMaxNodeKeys/32] masked-column bits
  static constexpr int kOffQrow = kOffMask + 4 * (kMaxNodeKeys / 32) * 4;   // int [2][2][128]
  static constexpr int kOffBar = kOffQrow + 4 * 128 * 4;
  static constexpr int kSBufs = 2;                    // S buffers per query tile
  // d = 64: the P V product is 80 columns wide - behind the 64 columns of V the B operand
  // continues in a slab of ones, so column 64 of O accumulates the sum of the bf16 weights that
  // normalises the row (the tensor pipe's floor per product does not depend on N up to 128, so
  // the extra columns are free and the softmax warps save one add per weight).  d = 128 would
  // pay for them (N = 144) and keeps the sum in registers.
  static constexpr bool kOnes = D == 64;
  static constexpr int kOCols = kOnes ? 80 : D;       // TMEM columns of one O accumulator
  static constexpr int kNumBar = 21 + 6 * NS + 12;
  static constexpr int kOffMisc = kOffBar + 8 * kNumBar;          // tmem slot, abort flag
  // Epilogue staging, one slice of 32 rows x kStageRow bytes per softmax warp: rows leave the
  // warp as whole 64- or 128-byte pieces instead of 16 bytes per lane and row.  d = 64: eight
  // slices of 4 KB.  d = 128 (less shared memory to spare): slices of 2 KB, those of query tile
  // 0 in the item's own key-row table, which nobody reads any more once the item's last K / V
  // tile has been issued and which is not rebuilt before the softmax warps release the set.
  static constexpr int kStageRow = (D == 64) ? 128 : 64;
  static constexpr int kStageWarp = 32 * kStageRow;
  static constexpr int kDescBytes = (sizeof(ItemDesc) + 15) / 16 * 16;
  static constexpr int kOffDesc = (kOffMisc + 16 + 15) / 16 * 16;   // ItemDesc [2], one per table set
  static constexpr int kOffStage = (kOffDesc + 2 * kDescBytes + 127) / 128 * 128;
  static constexpr int kOffOnes = (kOffStage + ((D == 64) ? 8 : 4) * kStageWarp + 1023) / 1024 * 1024;   // [TK keys x 128 B] of bf16 1.0
  static constexpr int kOffBias = kOnes ? kOffOnes + TK * 128 : kOffStage + ((D == 64) ? 8 : 4) * kStageWarp;   // float [2][kMaxWeightedSamples]: log2 weight of every sampled column (weighted sampling only)
  static constexpr int kTotal = kOffBias + 2 * kMaxWeightedSamples * 4;
  static_assert(kTotal <= 232448, "shared memory");
  static_assert(D == 64 || 4 * kStageWarp <= kMaxNodeKeys * 4, "staging of query tile 0 must fit one key-row table");
  static constexpr int kTmemCols = 512;
  static constexpr int kColO = 64 * 2 * kSBufs;       // S buffer b of tile i at 64 (kSBufs i + b); O_i at kColO + kOCols i
  static_assert(kColO + 2 * kOCols <= 512, "TMEM columns");
};

__device__ __forceinline__ void decode_pair(const AttnArgs& a, int pair, PairDesc& t, QTile& qa, QTile& qb) {
  const Geometry& g = a.g;
  t.partial = !a.direct;
  qa.valid = 1; qb.valid = 0;
  t.nbA = t.nbB = t.nsmp = 0;
  int s, q0n, k0n;
  if (pair < a.n_leaf_pairs) {
    // Leaf after leaf, the pairs of a leaf from the heaviest (last rows, most keys) to the lightest: items are
    // handed out in this order, so the CTAs that run at the same time work on a handful of neighbouring leaves
    // and find each other's K / V tiles in L2, and the list still ends with light items.
    const int uu = a.pairs_per_leaf - 1 - pair % a.pairs_per_leaf;
    const int rem = pair / a.pairs_per_leaf;
    t.seg = rem / a.leaves_per_seg;
    const int leaf = rem % a.leaves_per_seg;
    t.mode = 0; t.causal = a.dense_causal;
    // a leaf: the rows [k0, k0 + leaf) that exist; a non-causal call that is one block: all n queries against all nk keys
    t.k0 = leaf * g.leaf; t.nk = g.causal ? max(0, min(g.leaf, g.n - t.k0)) : g.nk;
    const int nq_leaf = g.causal ? t.nk : g.n;
    QTile* qs[2] = {&qa, &qb};
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int tt = 2 * uu + i;
      QTile& q = *qs[i];
      q.valid = tt < a.tiles_per_leaf && tt * kTileQ < nq_leaf;
      q.row0 = tt * kTileQ;
      q.q0 = t.k0 + tt * kTileQ;
      q.nq = min(kTileQ, nq_leaf - tt * kTileQ);
      const int lim = t.causal ? min(t.nk, q.row0 + q.nq) : t.nk;
      q.s1 = 0; q.n1 = q.valid ? (lim + TK - 1) / TK : 0; q.s2 = 0; q.n2 = 0;
    }
    t.orow_base = (size_t)t.seg * g.n; t.odelta = 0;
  } else {
    int level = 0;
    while (level + 1 < g.levels && pair >= a.level_pair_start[level + 1]) ++level;
    int idx = pair - a.level_pair_start[level];
    node_rows(g, level, 0, s, q0n, k0n);
    const int nodes_lvl = g.causal ? (1 << level) : 1;
    const int sorted = a.level_sorted[level];
    const int paired = a.level_paired[level];
    const int tiles_node = sorted ? node_blocks(s, g.b) * a.tiles_per_block : ((g.causal ? s : g.n) + kTileQ - 1) / kTileQ;
    const int pairs_node = paired ? (tiles_node + 1) / 2 : tiles_node;
    const int pn = idx % pairs_node; idx /= pairs_node;
    const int j = idx % nodes_lvl;
    t.seg = idx / nodes_lvl;
    node_rows(g, level, j, s, q0n, k0n);
    t.k0 = k0n; t.nk = s; t.qnode0 = q0n; t.causal = 0;
    t.nq_node = node_queries(g, s, q0n);
    t.bq = query_group(g.b, t.nq_node, s);
    t.mode = sorted;
    QTile* qs[2] = {&qa, &qb};
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int tn = paired ? 2 * pn + i : pn;
      QTile& q = *qs[i];
      q.valid = tn < tiles_node && (paired || i == 0);
      q.row0 = 0;
      if (sorted) {
        q.beta = tn / a.tiles_per_block;
        const int sub = tn % a.tiles_per_block;
        q.spos0 = q.beta * t.bq + sub * kTileQ;
        q.nq = t.bq > 0 ? min(kTileQ, block_len(t.nq_node, t.bq, q.beta) - sub * kTileQ) : 0;
        if (q.nq <= 0) q.valid = 0;                       // the group (a short last one, or one past the node's queries) has no such tile
        q.q0 = 0;
      } else {
        q.q0 = q0n + tn * kTileQ;
        q.nq = min(kTileQ, t.nq_node - tn * kTileQ);
        if (q.nq <= 0) q.valid = 0;
        q.s1 = 0; q.n1 = q.valid ? (s + TK - 1) / TK : 0; q.s2 = 0; q.n2 = 0;
      }
    }
    if (sorted) {
      t.slice = ((size_t)level * g.G + t.seg) * g.nl + (g.causal ? (size_t)j * s : 0);
      t.node = g.causal ? (1 << level) - 1 + j : 0;
      const int bt = (block_len(s, g.b, qa.beta) + TK - 1) / TK;                                  // key tiles of a block: its own length
      const int btb = qb.valid ? (block_len(s, g.b, qb.beta) + TK - 1) / TK : 0;
      t.nbA = bt;
      t.nbB = (qb.valid && qb.beta != qa.beta) ? btb : 0;
      t.nsmp = (g.m + TK - 1) / TK;
      // (a query tile that does not exist - the short last block may have fewer tiles - walks no key tiles)
      if (!qa.valid) { t.nbA = 0; t.nsmp = 0; }
      qa.s1 = 0; qa.n1 = t.nbA; qa.s2 = t.nbA + t.nbB; qa.n2 = t.nsmp;
      qb.s1 = t.nbB ? t.nbA : 0; qb.n1 = qb.valid ? (t.nbB ? btb : bt) : 0; qb.s2 = t.nbA + t.nbB; qb.n2 = qb.valid ? t.nsmp : 0;
    }
    if (a.direct) { t.orow_base = (size_t)t.seg * g.n; t.odelta = 0; }
    else { t.orow_base = (size_t)g.G * g.n + (size_t)level * g.G * g.nl + (size_t)t.seg * g.nl + (size_t)j * s; t.odelta = -q0n; }
  }
  t.ntiles = max(qa.s1 + qa.n1, max(qa.s2 + qa.n2, max(qb.s1 + qb.n1, qb.s2 + qb.n2)));
}

// a-th key tile of a query tile -> index in the pair's tile list
__device__ __forceinline__ int tile_of(const QTile& q, int a) { return a < q.n1 ? q.s1 + a : q.s2 + (a - q.n1); }
// GATHER_LATE: the softmax threads fetch the next item's Q tiles after, not before, they write
// the current item's results (see there).
// PRECISE: every softmax weight enters the P V product as a pair of bf16 numbers hi + lo (relative error
// 2^-17 instead of 2^-9): lo is written into the second half of the S buffer and multiplied by V with a
// second set of products.
// CAPPED: the sampled part of a sorted node's row sum carries the caps of Alg. 2 (lines 6, 7 and 9).
template <int D, bool GATHER_LATE, bool PRECISE, bool CAPPED>
__global__ void __launch_bounds__(384, 1) attn_tc_kernel(const __grid_constant__ AttnArgs a, const __grid_constant__ TmaMaps maps, int* status) {
  using C = Cfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr int MW = kMaxNodeKeys / 32;
  int* s_kidx_all = reinterpret_cast<int*>(smem + C::kOffIdx);              // [2][kMaxNodeKeys]
  uint32_t* s_mask_all = reinterpret_cast<uint32_t*>(smem + C::kOffMask);  // [2][2][MW]
  int* s_qrow_all = reinterpret_cast<int*>(smem + C::kOffQrow);             // [2][2][128]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);

  const uint32_t ubase = smem_u32(smem);
  const uint32_t bar0 = ubase + C::kOffBar;
  const uint32_t bar_q = bar0;                                                // Q tiles of the item landed
  const uint32_t bar_qfree = bar0 + 8;                                        // both issuers are done with Q
  auto bar_s = [&](int i, int b) { return bar0 + 168 + 8 * (6 * C::NS + 3 * i + b); };          // S_i buffer b written
  auto bar_p = [&](int i, int b) { return bar0 + 168 + 8 * (6 * C::NS + 6 + 3 * i + b); };      // P_i buffer b written
  auto bar_o = [&](int i) { return bar0 + 80 + 8 * i; };                      // O_i of the item complete
  auto bar_ofree = [&](int i) { return bar0 + 112 + 8 * i; };                 // O_i has been read out
  auto bar_tabfull = [&](int set) { return bar0 + 128 + 8 * set; };           // row tables of a set written
  auto bar_tabfree = [&](int set) { return bar0 + 144 + 8 * set; };           // softmax warps are done with a set
  auto bar_kfull = [&](int s) { return bar0 + 168 + 8 * s; };
  auto bar_vfull = [&](int s) { return bar0 + 168 + 8 * (C::NS + s); };
  auto bar_kempty = [&](int i, int s) { return bar0 + 168 + 8 * ((2 + i) * C::NS + s); };     // released by issuer i
  auto bar_vempty = [&](int i, int s) { return bar0 + 168 + 8 * ((4 + i) * C::NS + s); };

  const Geometry& g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HA_T0(t_cta);

  // A CTA of a launch in which some wait already timed out returns at once (nothing allocated
  // yet), so a stuck launch drains quickly instead of timing out tile after tile.
  if (tid == 0) *s_abort = *reinterpret_cast<volatile int*>(status);
  __syncthreads();
  if (*s_abort) return;
  __syncthreads();

  // ---- setup: barriers, TMEM ---------------------------------------------------------------------
  if (tid == 0) {
    mbar_init(bar_q, 32 + 256);                         // item preparer + softmax threads
    mbar_init(bar_qfree, 2);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_o(i), 1);
      mbar_init(bar_ofree(i), 128);
      mbar_init(bar_tabfull(i), 1);
      mbar_init(bar_tabfree(i), 257);                   // 256 softmax threads + the K / V streamer
      for (int b = 0; b < C::kSBufs; ++b) { mbar_init(bar_s(i, b), 1); mbar_init(bar_p(i, b), 128); }
    }
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(bar_kfull(s), 32);
      mbar_init(bar_vfull(s), 32);
      for (int i = 0; i < 2; ++i) { mbar_init(bar_kempty(i, s), 1); mbar_init(bar_vempty(i, s), 1); }
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if constexpr (C::kOnes) {
    for (int k = tid; k < TK * 128 / 16; k += 384) *reinterpret_cast<uint4*>(smem + C::kOffOnes + 16 * k) = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);
    fence_async_smem();                                 // the tensor pipe reads the slab through the async proxy
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // The CTA is persistent: it walks over work items (pairs of query tiles) blockIdx.x,
  // blockIdx.x + gridDim.x, ...  Every role runs the same item loop at its own pace; what
  // they hand to each other across items is described at the barriers above.  All phase
  // counters keep running across items.
  if (warp < 8) {
    // ================= softmax + epilogue of query tile i: thread = query row ==================
    const int i = warp >> 2;
    const int row = tid & 127;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t colO = C::kColO + C::kOCols * i;
    int ga = 0;                                       // key tiles this warpgroup has processed so far (all items)
    int gbase = 0;                                    // global index (all items) of the item's first key tile
    int vi = 0;                                       // items in which this query tile existed
    bool ok = true;
    int it = 0;
    // Gathered Q tiles (sorted rows) are fetched by the 256 softmax threads together, 16-byte
    // chunks through cp.async: one warp alone is limited by the copies it can keep in flight.
    // Thread -> column chunk cq of rows rq0, rq0 + 256 / CPR, ...; its arrival on the Q barrier
    // is attached to its copies.  (Tiles of consecutive rows are one TMA box, issued by the
    // item preparer; then the arrival here is immediate.)
    auto gather_q = [&](int nit) {
      bool good = mbar_wait<20, 19>(bar_tabfull(nit & 1), (nit >> 1) & 1, s_abort, status);
      if (!good) return false;
      const ItemDesc& de = *reinterpret_cast<const ItemDesc*>(smem + C::kOffDesc + (nit & 1) * C::kDescBytes);
      const PairDesc& t = de.t;
      if (t.mode < 0) return true;                        // the end of the work list: nothing to fetch
      if (nit >= 1) good = mbar_wait<20, 20>(bar_qfree, (nit - 1) & 1, s_abort, status);
      if (!good) return false;
      const QTile &qa = de.qa, &qb = de.qb;
      if (t.mode == 1) {
        constexpr int CPR = D / 8;
        constexpr int RS = 256 / CPR;                       // rows covered by the 256 threads per step
        const int cq = tid % CPR, rq0 = tid / CPR;
        const char* qsrc = reinterpret_cast<const char*>(a.q) + (size_t)t.seg * g.n * (D * 2) + cq * 16;
        const int* rows = s_qrow_all + (nit & 1) * 2 * 128;
#pragma unroll
        for (int ti = 0; ti < 2; ++ti) {
          if (!(ti ? qb.valid : qa.valid)) continue;       // nobody reads the tile of a query tile that does not exist
          int v[128 / RS];
#pragma unroll
          for (int k = 0; k < 128 / RS; ++k) v[k] = rows[ti * 128 + rq0 + k * RS];
#pragma unroll
          for (int k = 0; k < 128 / RS; ++k)               // padding rows: the segment's first row (results never stored)
            cp_async16(ubase + C::kOffQ + ti * C::kQTile + tile_off<128>(rq0 + k * RS, cq), qsrc + (size_t)(uint32_t)max(v[k], 0) * (D * 2));
        }
        cp_async_arrive_noinc(bar_q);
      } else {
        mbar_arrive(bar_q);
      }
      return true;
    };
    HA_LDECL(a_tab); HA_LDECL(a_ws); HA_LDECL(a_cmp); HA_LDECL(a_epi); HA_LDECL(a_gq); HA_LDECL(a_bo); HA_LDECL(a_tiles); HA_LDECL(a_ws0); HA_LDECL(a_c1); HA_LDECL(a_c2); HA_LDECL(a_c3); HA_LDECL(a_c4); HA_LDECL(a_e1); HA_LDECL(a_e2); HA_LDECL(a_e3);
    HA_T0(t_role);
    ok = __all_sync(0xffffffffu, gather_q(0));
    for (; ok; ++it) {
      const int set = it & 1;
      const uint32_t* s_mask = s_mask_all + (set * 2 + i) * MW;
      const int* s_qrow = s_qrow_all + (set * 2 + i) * 128;
      // the tables of this item (also for a warpgroup without a tile: it may not run ahead)
      HA_T0(tt);
      ok = __all_sync(0xffffffffu, mbar_wait<20, 14>(bar_tabfull(set), (it >> 1) & 1, s_abort, status));
      if (!ok) break;
      HA_LACC(a_tab, tt);
      const ItemDesc& de = *reinterpret_cast<const ItemDesc*>(smem + C::kOffDesc + set * C::kDescBytes);
      const PairDesc t = de.t;
      if (t.mode < 0) break;                              // the work list is exhausted
      const QTile q = i ? de.qb : de.qa;
      const int total = q.n1 + q.n2;
      const float wlog = (t.mode == 1 && g.m > 0) ? log2f((float)t.nk / (float)g.m) : 0.f;   // log2(N/m): weight of a sampled column
      // key tiles of this item with masked columns for this query tile, one bit per tile (an item has at most 32)
      unsigned tile_masked = 0;
      if (t.mode == 1) tile_masked = __ballot_sync(0xffffffffu, lane < t.ntiles && (s_mask[2 * lane] | s_mask[2 * lane + 1]) != 0);
      float m_ref = -INFINITY;
      uint64_t l01 = 0;             // l: unrounded row sum (two partial sums, packed)
      float lra = 0.f, lrb = 0.f;   // lr: sum of the bf16 weights (two partial sums; the mixed-precision add takes the bf16 halves as they are)
      // Alg. 2 with caps (sorted nodes only): the masked row sum (block part) is complete when the first
      // sampled tile starts; from then on every sampled weight enters the row sum as min(weight, (N/m) C_i),
      // C_i = cap_scale m / (N ln N) (masked_i + tau / kappa), while the numerator keeps the weight itself.
      const bool capped_item = CAPPED && t.mode == 1 && g.m > 0 && a.capped;
      float lblk = 0.f;             // masked row sum in units of 2^m_ref
      bool in_samples = false;
      float capfac = 0.f, lfloor = -INFINITY;     // (N/m) cap_scale m / (N ln N); log2(tau / kappa)
      // weighted sampling (columns drawn by value norms): every sampled column carries its own log2 weight
      const bool weighted_item = CAPPED && t.mode == 1 && a.sample_wlog != nullptr;
      const float* s_bias = reinterpret_cast<const float*>(smem + C::kOffBias) + set * kMaxWeightedSamples;
      if (capped_item) {
        capfac = a.cap_scale / (logf((float)t.nk));
        lfloor = a.ltau[(size_t)t.seg * g.nodes + t.node] - a.log2_kappa;
      }
      for (int na = 0; na < total && ok; ++na) {
        const int j = tile_of(q, na);
        const int gw = ga + na;
        const int buf = gw % C::kSBufs;
        HA_T0(tw);
        ok = __all_sync(0xffffffffu, mbar_wait<20, 2>(bar_s(i, buf), (gw / C::kSBufs) & 1, s_abort, status));   // warp-uniform: TMEM ops are .aligned
        if (!ok) break;
        HA_LACC(a_ws, tw);
#ifdef HA_TC_TIMING
        if (na == 0) a_ws0 += clock64() - tw;
#endif
        HA_T0(tc);
        tc_fence_after();
        // mask kind of this (query tile, key tile): uniform over the warpgroup
        const bool table = (tile_masked >> j) & 1u;
        // (weighted sampling: the tile's columns have weights of their own; the largest one stands in where one number is needed)
        const bool weighted_tile = weighted_item && j >= t.nbA + t.nbB;
        const float ubias = (t.mode == 1 && j >= t.nbA + t.nbB) ? (weighted_tile ? t.bias_max : wlog) : 0.f;
        const bool dense_mask = t.mode != 1 && ((j * TK + TK > t.nk) || (t.causal && j * TK + TK - 1 > q.row0));
        // The 64 scores of this row are read from TMEM once; then (1) the row maximum, (2)
        // exponentials, row sums and the bf16 P written over the first half of the S buffer.
        // The reference maximum only moves when the tile exceeds it by more than 2^32, and then
        // by a whole number of octaves, so that what is already accumulated (O and the row
        // sums) is rescaled exactly.
        uint32_t ra[32], rb[32];
        const uint32_t sbase = lane_addr + 64 * (C::kSBufs * i + buf);
        // masked columns become -inf before the tile is read (out of line, in TMEM): they then
        // drop out of the maximum and exponentiate to zero without any test in this loop
        if (table || dense_mask) {
          uint32_t visa, visb;
          if (table) { visa = ~s_mask[j * 2]; visb = ~s_mask[j * 2 + 1]; }
          else {
            const int climit = t.causal ? min(t.nk - 1, q.row0 + row) : t.nk - 1;   // last visible column of this row
            const int rel = climit - j * TK;            // columns 0..rel of the tile are visible
            visa = rel >= 31 ? 0xffffffffu : (rel < 0 ? 0u : ((2u << rel) - 1u));
            visb = rel >= 63 ? 0xffffffffu : (rel < 32 ? 0u : ((2u << (rel - 32)) - 1u));
          }
          mask_scores(sbase, visa, visb);
        }
        // The second half of the scores is requested once the first has arrived and lands while
        // the first is exponentiated.
        tmem_ld32_issue(sbase, ra);
        tmem_ld32_wait(ra);
        tmem_ld32_issue(sbase + 32, rb);
        HA_LACC(a_c1, tc);
        // The row maximum is NOT computed per tile.  Any reference within a few dozen octaves of the
        // true maximum serves (the accumulators are fp32 and the weights keep their relative
        // precision as bf16), so a tile is exponentiated against the reference the row already
        // has, and only when the tile's sum of weights shows that some score lay more than ~2^34
        // above it (or the row has no reference yet: first tile of an item) is the maximum
        // taken, the reference moved by whole octaves, O rescaled exactly, and the tile
        // exponentiated again from the scores still held in registers.
        auto move_reference = [&]() -> bool {
          tmem_ld32_wait(rb);
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            m0 = max3(m0, __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
            m1 = max3(m1, __uint_as_float(ra[e + 2]), __uint_as_float(ra[e + 3]));
            m2 = max3(m2, __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
            m3 = max3(m3, __uint_as_float(rb[e + 2]), __uint_as_float(rb[e + 3]));
          }
          m0 = fmaxf(m0, m2); m1 = fmaxf(m1, m3);
          const float xm = fmaf(fmaxf(m0, m1), a.scale_log2, ubias);   // scale_log2 > 0: the maximum commutes with it
          const bool grow = xm > m_ref + kRescaleThreshold;
          if (!__any_sync(0xffffffffu, grow)) return true;
          float alpha = 1.f;
          if (grow) {
            // first tile: leave head room for the weight log2(N/m) that the sampled columns will
            // add, so that reaching them does not move the reference again (any reference within
            // 2^32 below the true maximum serves; a higher one only shifts the exponents)
            if (m_ref == -INFINITY) { m_ref = xm + (wlog - ubias); alpha = 0.f; }
            else { const float k = ceilf(xm - m_ref); m_ref += k; alpha = ex2(-k); }
          }
          { const uint64_t al2 = pack_f2(alpha, alpha); l01 = fmul2(l01, al2); lra *= alpha; lrb *= alpha; lblk *= alpha; }
          // O may only be touched between two PV products: the one of the previous tile must
          // have finished (the one of this tile cannot start before this tile's P is published)
          // That product's completion is what releases its V stage to the streamer, so the
          // stage's barrier tells (the issuer has nothing extra to commit for this rare path).  Its
          // phase cannot run ahead of this warpgroup: the next product on the same stage is NS key
          // tiles later and needs this warpgroup's P first.
          if (na > 0) {
            const int gjp = gbase + tile_of(q, na - 1);
            if (!__all_sync(0xffffffffu, mbar_wait<20, 3>(bar_vempty(i, gjp % C::NS), (gjp / C::NS) & 1, s_abort, status))) return false;
            tc_fence_after();
            rescale_row(lane_addr + colO, C::kOCols, alpha);
          }
          return true;
        };
        if (__any_sync(0xffffffffu, m_ref == -INFINITY)) {
          ok = move_reference();
          if (!ok) break;
        }
        const bool capped_tile = capped_item && j >= t.nbA + t.nbB;
        if (capped_tile && !in_samples) {            // the block part is complete: its row sum is the masked sum of line 6
          float b0, b1;
          unpack_f2(l01, b0, b1);
          lblk = b0 + b1;
          in_samples = true;
        }
        const uint64_t sc2 = pack_f2(a.scale_log2, a.scale_log2);
        uint64_t lt2;               // this tile's unrounded sum of weights (two partial sums, packed)
        float lrta, lrtb;           // this tile's sum of the bf16 weights (d = 128)
        for (int attempt = 0;; ++attempt) {
          const float off = ubias - (m_ref == -INFINITY ? 0.f : m_ref);
          // packed fp32 arithmetic (two lanes per instruction) for the scaling and the row sums
          const uint64_t off2 = pack_f2(off, off);
          lt2 = 0; lrta = 0.f; lrtb = 0.f;
          auto chunk_exp = [&](const uint32_t (&r)[32], int c) {
            uint32_t p[16], plo[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              float x0, x1;
              unpack_f2(ffma2(pack_u2(r[e], r[e + 1]), sc2, off2), x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              lt2 = fadd2(lt2, pack_f2(p0, p1));
              const uint32_t w = pack2(p0, p1);
              if constexpr (!C::kOnes)
                asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}" : "+f"(lrta), "+f"(lrtb) : "r"(w));
              p[e >> 1] = w;
              if constexpr (PRECISE) {
                // what the rounding to bf16 left over, as a second bf16 number (infinite weights leave none)
                const float r0 = p0 - __uint_as_float(w << 16), r1 = p1 - __uint_as_float(w & 0xffff0000u);
                const uint32_t wl = pack2(r0 == r0 ? r0 : 0.f, r1 == r1 ? r1 : 0.f);
                if constexpr (!C::kOnes)
                  asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}" : "+f"(lrta), "+f"(lrtb) : "r"(wl));
                plo[e >> 1] = wl;
              }
            }
            tmem_st16(sbase + c * 16, p);
            if constexpr (PRECISE) {
              tmem_st16(sbase + 32 + c * 16, plo);
            }
          };
          // capped tiles: the row sum takes min(weight, cap), the check below and P take the weight itself
          uint64_t ltu2 = 0;
          const float capw = capped_tile ? capfac * (lblk + (m_ref == -INFINITY ? 0.f : ex2(lfloor - m_ref))) : 0.f;
          auto chunk_exp_capped = [&](const uint32_t (&r)[32], int c) {
            uint32_t p[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              float x0, x1;
              unpack_f2(ffma2(pack_u2(r[e], r[e + 1]), sc2, off2), x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              ltu2 = fadd2(ltu2, pack_f2(p0, p1));
              lt2 = fadd2(lt2, pack_f2(fminf(p0, capw), fminf(p1, capw)));
              p[e >> 1] = pack2(p0, p1);
            }
            tmem_st16(sbase + c * 16, p);
          };
          // weighted tiles: x = score * scale + (the column's log2 weight - reference)
          const float* bias_tile = s_bias + (j - (t.nbA + t.nbB)) * TK;
          const uint64_t nref2 = pack_f2(off - ubias, off - ubias);
          auto chunk_exp_weighted = [&](const uint32_t (&r)[32], int c) {
            uint32_t p[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float2 bb = *reinterpret_cast<const float2*>(bias_tile + c * 32 + e);
              float x0, x1;
              unpack_f2(ffma2(pack_u2(r[e], r[e + 1]), sc2, fadd2(pack_f2(bb.x, bb.y), nref2)), x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              lt2 = fadd2(lt2, pack_f2(p0, p1));
              const uint32_t w = pack2(p0, p1);
              if constexpr (!C::kOnes)
                asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}" : "+f"(lrta), "+f"(lrtb) : "r"(w));
              p[e >> 1] = w;
            }
            tmem_st16(sbase + c * 16, p);
          };
          HA_T0(tc2);
          if constexpr (PRECISE) tmem_ld32_wait(rb);     // the lo halves overwrite the second half of the scores
          if (CAPPED && capped_tile) chunk_exp_capped(ra, 0); else if (CAPPED && weighted_tile) chunk_exp_weighted(ra, 0); else chunk_exp(ra, 0);
          HA_LACC(a_c2, tc2);
          HA_T0(tc3);
          tmem_ld32_wait(rb);
          if (CAPPED && capped_tile) chunk_exp_capped(rb, 1); else if (CAPPED && weighted_tile) chunk_exp_weighted(rb, 1); else chunk_exp(rb, 1);
          HA_LACC(a_c3, tc3);
          float lt0, lt1;
          unpack_f2((CAPPED && capped_tile) ? ltu2 : lt2, lt0, lt1);
          // (the negated comparison also catches an infinite sum; one second attempt at most: after the
          // reference has moved every finite score is within range, and non-finite inputs must not loop)
          if (attempt == 1 || !__any_sync(0xffffffffu, !(lt0 + lt1 <= kTileSumLimit))) break;
          ok = move_reference();
          if (!ok) break;
        }
        if (!ok) break;
        HA_T0(tc4);
        l01 = fadd2(l01, lt2);
        lra += lrta; lrb += lrtb;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p(i, buf));
        HA_LACC(a_c4, tc4);
        HA_LACC(a_cmp, tc);
#ifdef HA_TC_TIMING
        a_tiles += 1;
#endif
      }
      if (!ok) break;
      // The next item's Q tiles go out before this item's results are written, so that they are
      // there when the results are - except for fp32 partial results of d = 128 (causal
      // recursion): those are twice the bytes to stage and store and queue behind the gather's
      // copies in the load/store unit (measured: 5 % faster with the gather after them, while
      // bf16 results are 5 % slower that way).
      HA_T0(tg);
      if (!GATHER_LATE) {
        ok = __all_sync(0xffffffffu, gather_q(it + 1));
        if (!ok) break;
      }
      HA_LACC(a_gq, tg);
      HA_T0(te);
      // epilogue: normalise, log-sum-exp, rows back to their original places
      if (q.valid) {
        ok = __all_sync(0xffffffffu, mbar_wait<20, 5>(bar_o(i), vi & 1, s_abort, status));
        if (!ok) break;
        HA_LACC(a_bo, te);
        tc_fence_after();
        const int qr = s_qrow[row];
        float l0, l1, lr0, lr1;
        unpack_f2(l01, l0, l1);
        lr0 = lra; lr1 = lrb;
        if constexpr (C::kOnes) {                       // the sum of the bf16 weights sits in column D of O
          uint32_t sumw;
          asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n\ttcgen05.wait::ld.sync.aligned;\n" : "=r"(sumw) : "r"(lane_addr + colO + D) : "memory");
          lr0 = __uint_as_float(sumw); lr1 = 0.f;
        }
        float inv = 1.f / (lr0 + lr1);
        float lse = (m_ref + log2f(l0 + l1)) * 0.69314718055994531f;
        if (capped_item) {
          // line 9: d~_i = masked_i + max(d_i, tau / kappa), d_i the sum of the capped sampled weights
          if (!in_samples) lblk = l0 + l1;
          const float fl = m_ref == -INFINITY ? 0.f : ex2(lfloor - m_ref);
          const float dt = lblk + fmaxf((l0 + l1) - lblk, fl);
          inv = 1.f / dt;
          lse = (m_ref + log2f(dt)) * 0.69314718055994531f;
        }
        const size_t orow = t.orow_base + (size_t)(qr + t.odelta);
        {
          // O leaves TMEM in pieces of 16 columns (thread = row), is normalised (and rounded to
          // bf16 for a bf16 result) and staged in shared memory, XOR-swizzled so that neither
          // side has bank conflicts; then LPR lanes per row write kStageRow contiguous bytes of
          // RPI rows per instruction.
          constexpr int RB = C::kStageRow;
          constexpr int LPR = RB / 16, RPI = 32 / LPR, NI = 32 / RPI;
          constexpr int NP = D / 16;
          const bool f32o = t.partial ? !a.part_bf16 : a.out_fp32;
          char* obase = reinterpret_cast<char*>(t.partial ? a.part_o : a.out);
          const long long myoff = qr >= 0 ? (long long)(orow * (size_t)(D * (f32o ? 4 : 2))) : -1;
          long long roff[NI];
#pragma unroll
          for (int k = 0; k < NI; ++k) roff[k] = __shfl_sync(0xffffffffu, myoff, RPI * k + lane / LPR);
          const uint32_t stg = (D == 64) ? ubase + C::kOffStage + warp * C::kStageWarp
                             : (i == 0 ? ubase + C::kOffIdx + set * (kMaxNodeKeys * 4) : ubase + C::kOffStage) + (warp & 3) * C::kStageWarp;
          const int xw = (RB == 128) ? (lane & 7) : ((lane >> 1) & 3);       // swizzle of this thread's own row
          const int crow = lane / LPR, cc = lane % LPR;
          const int lg_pps = f32o ? (RB == 128 ? 1 : 0) : (RB == 128 ? 2 : 1);   // log2(pieces per staging step)
          uint32_t r[16];
          HA_LACC(a_e1, te);
          tmem_ld16_issue(lane_addr + colO, r);
#pragma unroll 1
          for (int pc = 0; pc < NP; ++pc) {
            HA_T0(te2);
            tmem_ld16_wait(r);
            float f[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) f[e] = __uint_as_float(r[e]) * inv;
            if (pc + 1 < NP) tmem_ld16_issue(lane_addr + colO + (pc + 1) * 16, r);
            else { tc_fence_before(); mbar_arrive(bar_ofree(i)); }           // O has been read: the next item may overwrite it
            const int pin = pc & ((1 << lg_pps) - 1);
            const uint32_t srow = stg + lane * RB;
            if (f32o) {
#pragma unroll
              for (int c = 0; c < 4; ++c)
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(srow + (((pin * 4 + c) ^ xw) << 4)),
                             "f"(f[4 * c]), "f"(f[4 * c + 1]), "f"(f[4 * c + 2]), "f"(f[4 * c + 3]) : "memory");
            } else {
#pragma unroll
              for (int c = 0; c < 2; ++c)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(srow + (((pin * 2 + c) ^ xw) << 4)),
                             "r"(pack2(f[8 * c], f[8 * c + 1])), "r"(pack2(f[8 * c + 2], f[8 * c + 3])),
                             "r"(pack2(f[8 * c + 4], f[8 * c + 5])), "r"(pack2(f[8 * c + 6], f[8 * c + 7])) : "memory");
            }
            HA_LACC(a_e2, te2);
            if (pin == (1 << lg_pps) - 1) {
              HA_T0(te3);
              __syncwarp();
              const int step = pc >> lg_pps;
#pragma unroll
              for (int k = 0; k < NI; ++k) {
                const int rw = RPI * k + crow;
                const int xr = (RB == 128) ? (rw & 7) : ((rw >> 1) & 3);
                uint4 w;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                             : "r"(stg + rw * RB + ((cc ^ xr) << 4)) : "memory");
                if (roff[k] >= 0) *reinterpret_cast<uint4*>(obase + roff[k] + step * RB + cc * 16) = w;
              }
              __syncwarp();
              HA_LACC(a_e3, te3);
            }
          }
        }
        if (qr >= 0) {
          if (t.partial) a.part_lse[orow] = lse;
          else a.lse[orow] = lse;
        }
        ++vi;
      }
      if (GATHER_LATE) {
        ok = __all_sync(0xffffffffu, gather_q(it + 1));
        if (!ok) break;
      }
      mbar_arrive(bar_tabfree(set));
      HA_LACC(a_epi, te);
      ga += total;
      gbase += t.ntiles;
    }
#ifdef HA_TC_TIMING
    if (row == 0 && i == 0) {
      HA_LFLUSH(9, a_tab); HA_LFLUSH(0, a_ws); HA_LFLUSH(2, a_cmp); HA_LFLUSH(15, a_epi); HA_LFLUSH(16, a_gq); HA_LFLUSH(17, a_bo);
      HA_LFLUSH(20, a_tiles); HA_TACC(18, t_role); HA_LFLUSH(19, it);
      HA_LFLUSH(40, a_e1); HA_LFLUSH(41, a_e2); HA_LFLUSH(42, a_e3); HA_LFLUSH(24, a_ws0); HA_LFLUSH(22, a_c1); HA_LFLUSH(29, a_c2); HA_LFLUSH(30, a_c3); HA_LFLUSH(31, a_c4);
    }
#endif
  } else if (warp < 10) {
    // ================= MMA issue: one lane per query tile (warp 8: tile 0, warp 9: tile 1) ===========
    // Each issuer walks its own key tiles: scores run two tiles ahead of the PV products
    // (S buffers alternate).  A tcgen05.mma occupies the issuing thread and the tensor pipe
    // for about 55-65 cycles whatever its size, so the two chains are issued by two threads.
    // The issuer shares its scheduler with two busy softmax warps and has no instruction-level
    // parallelism of its own, so its loop is kept to a minimum of instructions: descriptors
    // are two 32-bit words of which only the low one moves, waits are one probe in the common
    // case, everything unusual lives in out-of-line slow paths.
    const int i = warp - 8;
    if (lane == 0) {
      constexpr uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)TK >> 3) << 17) | ((128u >> 4) << 24);
      constexpr uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)C::kOCols >> 3) << 17) | ((128u >> 4) << 24);
      // descriptor: low word = start address >> 4 | (leading byte offset >> 4) << 16,
      // high word = stride byte offset >> 4 | version 1 << 14 | 128-byte swizzle 2 << 29
      constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t dq_lo = ((ubase + C::kOffQ + i * C::kQTile) >> 4) | (1u << 16);
      const uint32_t dk_lo0 = ((ubase + C::kOffK) >> 4) | (1u << 16);
      // V descriptors: the leading byte offset is the distance to the next 64 columns of the B
      // operand - the tile's second slab (d = 128) or the slab of ones (d = 64), whose distance
      // shrinks by one tile per stage
      const uint32_t dv_lo0 = ((ubase + C::kOffV) >> 4) | (((uint32_t)(C::kOnes ? C::kOffOnes - C::kOffV : TK * 128) >> 4) << 16);
      constexpr uint32_t dv_step = (uint32_t)(C::kTile >> 4) - (C::kOnes ? ((uint32_t)(C::kTile >> 4) << 16) : 0u);   // per stage
      const uint32_t ocol = tmem + C::kColO + C::kOCols * i;
      const uint32_t scol = tmem + 64 * C::kSBufs * i;
      bool ok = true;
      int gbase = 0;                        // global index (all items) of the item's first key tile
      int knext = 0, vnext = 0;             // next global tile whose K / V stage this issuer has to observe and release
      int ga = 0;                           // key tiles issued so far for this query tile (all items)
      int vi = 0;                           // items in which this query tile existed
      // Tiles this query tile does not look at (the other tile's own block, or everything when
      // the tile does not exist) are released when the walk passes them, but only after they
      // have arrived: a release must never overtake the loader's wait for the previous
      // release of the same stage (the barrier would wrap around unseen).  Releases go through
      // tcgen05.commit, so they also stay behind this thread's earlier MMAs.
      auto skip_k = [&](int gj) {
        for (; knext < gj && ok; ++knext) {
          ok = wait_fast<7>(bar_kfull(knext % C::NS), (knext / C::NS) & 1, s_abort, status);
          if (ok) umma_commit(bar_kempty(i, knext % C::NS));
        }
      };
      auto skip_v = [&](int gj) {
        for (; vnext < gj && ok; ++vnext) {
          ok = wait_fast<9>(bar_vfull(vnext % C::NS), (vnext / C::NS) & 1, s_abort, status);
          if (ok) umma_commit(bar_vempty(i, vnext % C::NS));
        }
      };
      int it = 0;
      HA_LDECL(b_q); HA_LDECL(b_p); HA_LDECL(b_v); HA_LDECL(b_k);
      HA_T0(tloop);
      for (; ok; ++it) {
        ok = wait_fast<22>(bar_tabfull(it & 1), (it >> 1) & 1, s_abort, status);
        if (!ok) break;
        const ItemDesc& de = *reinterpret_cast<const ItemDesc*>(smem + C::kOffDesc + (it & 1) * C::kDescBytes);
        if (de.t.mode < 0) break;
        const QTile q = i ? de.qb : de.qa;
        const int total = q.n1 + q.n2;
        const int ntiles = de.t.ntiles;
#ifdef HA_TC_TIMING
        if (i == 0) atomicAdd(&g_tc_timing[14], (unsigned long long)ntiles);
#endif
        // Q of this item (an issuer without a tile waits too: it may not run ahead of the others)
        HA_T0(tq);
        ok = wait_fast<6>(bar_q, it & 1, s_abort, status);
        if (!ok) break;
        HA_LACC(b_q, tq);
        fence_async_smem();
        if (total == 0) mbar_arrive(bar_qfree);
        auto issue_pv = [&](int a2) {
          // ---- O += P V of key tile a2 ----------------------------------------------------------
          const int gj = gbase + tile_of(q, a2);
          const int s = gj % C::NS;
          const int gw = ga + a2;
          if (gj != vnext) skip_v(gj);
          HA_T0(tp);
          ok = ok && wait_fast<8>(bar_p(i, gw % C::kSBufs), (gw / C::kSBufs) & 1, s_abort, status);
          HA_LACC(b_p, tp);
          HA_T0(tv);
          ok = ok && wait_fast<9>(bar_vfull(s), (gj / C::NS) & 1, s_abort, status);
          HA_LACC(b_v, tv);
          // the first product of an item overwrites O: the previous item's O must have been read
          if (a2 == 0 && vi > 0) ok = ok && wait_fast<15>(bar_ofree(i), (vi - 1) & 1, s_abort, status);
          if (!ok) return;
          fence_async_smem();
          tc_fence_after();
          const uint32_t pcol = scol + 64 * (gw % C::kSBufs);
          const uint32_t dv_lo = dv_lo0 + (uint32_t)s * dv_step;
          mma_ts2(ocol, pcol, dv_lo, desc_hi, idesc_o, a2 > 0);
#pragma unroll
          for (int kk = 1; kk < TK / 16; ++kk) mma_ts2(ocol, pcol + kk * 8, dv_lo + kk * (2048 >> 4), desc_hi, idesc_o, 1);
          if constexpr (PRECISE) {
#pragma unroll
            for (int kk = 0; kk < TK / 16; ++kk) mma_ts2(ocol, pcol + 32 + kk * 8, dv_lo + kk * (2048 >> 4), desc_hi, idesc_o, 1);
          }
          umma_commit(bar_vempty(i, s));
          vnext = gj + 1;
          if (a2 == total - 1) umma_commit(bar_o(i));
        };
        auto issue_s = [&](int r) {
          // ---- S = Q K^T of key tile r into buffer (ga + r) % kSBufs --------------------------------
          const int gj = gbase + tile_of(q, r);
          const int s = gj % C::NS;
          const int gw = ga + r;
          if (gj != knext) skip_k(gj);
          HA_T0(tk);
          ok = ok && wait_fast<7>(bar_kfull(s), (gj / C::NS) & 1, s_abort, status);
          HA_LACC(b_k, tk);
          if (!ok) return;
          fence_async_smem();
          tc_fence_after();
          const uint32_t dcol = scol + 64 * (gw % C::kSBufs);
          const uint32_t dk_lo = dk_lo0 + (uint32_t)s * (C::kTile >> 4);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            mma_ss2(dcol, dq_lo + (((ks >> 2) * (128 * 128) + (ks & 3) * 32) >> 4),
                    dk_lo + (((ks >> 2) * (TK * 128) + (ks & 3) * 32) >> 4), desc_hi, idesc_s, ks > 0);
          umma_commit(bar_s(i, gw % C::kSBufs));
          umma_commit(bar_kempty(i, s));
          knext = gj + 1;
          if (r == total - 1) umma_commit(bar_qfree);     // nothing of this item reads Q any more
        };
        // The S buffer of tile r held P of tile r - kSBufs, so the product P V of that tile must be
        // issued before the scores of tile r.  Two buffers: P V (r - 2), then S (r).  Three: the
        // scores go first - they do not wait for the warpgroup - and are ready a tile earlier.
        for (int r = 0; r < total + 2 && ok; ++r) {
          if (C::kSBufs == 2) {
            if (r >= 2) issue_pv(r - 2);
            if (ok && r < total) issue_s(r);
          } else {
            if (r < total) issue_s(r);
            if (ok && r >= 2) issue_pv(r - 2);
          }
        }
        if (!ok) break;
        // what is left of the item's tiles (all of them for a query tile that does not exist) is
        // released K, V, K, V ... like the streamer fills them: releasing all K tiles first would
        // wait for a K tile whose stage the streamer cannot reach before a V tile is released
        for (int e = min(knext, vnext) + 1; e <= gbase + ntiles && ok; ++e) { skip_k(e); skip_v(e); }
        gbase += ntiles;
        ga += total;
        vi += q.valid;
      }
      if (i == 0) { HA_TACC(8, tloop); HA_TACC(12, t_cta); HA_LFLUSH(7, b_q); HA_LFLUSH(4, b_p); HA_LFLUSH(5, b_v); HA_LFLUSH(6, b_k); }
#ifdef HA_TC_TIMING
      if (i == 0) atomicAdd(&g_tc_timing[13], 1ull);
#endif
    }
    __syncwarp();
  } else if (warp == 10) {
    // ================= item preparer: row tables of an item, then its Q tiles ========================
    // Runs one item ahead of the K / V streamer where it can: a table set becomes free when the
    // softmax warps and the streamer are done with the item before the previous one, so the
    // dependent global lookups below overlap with the computation of the item in between.
    bool ok = true;
    int it = 0;
    for (; ok; ++it) {
      HA_T0(tdec);
      // Work items are handed out by a counter in global memory, in list order (heavy first): whichever CTA
      // is free takes the next one.
      int item = 0;
      if (lane == 0) item = atomicAdd(a.sched, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      const bool end = item >= a.total_pairs;
      PairDesc t = {}; QTile qa = {}, qb = {};
      if (!end) decode_pair(a, item, t, qa, qb);
      else t.mode = -1;                                   // tells every role that the list is exhausted
      if (lane == 0) HA_TACC(26, tdec);
      const int set = it & 1;
      int* s_kidx = s_kidx_all + set * kMaxNodeKeys;
      uint32_t* s_mask = s_mask_all + set * 2 * MW;
      int* s_qrow = s_qrow_all + set * 2 * 128;
      HA_T0(ttab);
      if (it >= 2) {
        ok = mbar_wait<100, 16>(bar_tabfree(set), ((it >> 1) - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      if (lane == 0) HA_TACC(21, ttab);
      if (lane == 0) {
        ItemDesc* de = reinterpret_cast<ItemDesc*>(smem + C::kOffDesc + set * C::kDescBytes);
        de->t = t; de->qa = qa; de->qb = qb;
      }
      if (end) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tabfull(set));
        break;
      }
      const int segrow = t.seg * g.n;                       // row coordinate of the segment's first query row ...
      const int segrow_k = t.seg * g.nk;                    // ... and of its first key row
      // Key rows as tensor-map row coordinates.  Every global load of a batch is issued before
      // the first one is used; the warp covers 32 consecutive columns per step, so one ballot
      // yields a whole word of the mask tables.  Padding columns point at a valid row (they are
      // masked, so that row only has to be finite) and are masked for both tiles.
      if (t.mode == 1) {
        constexpr int UB = 8;
        const int bcols = t.nbA * TK;
        const int nblk = (t.nbA + t.nbB) * TK;            // columns of the block part (multiple of 64)
        const int ncols = t.ntiles * TK;
        const int32_t* smp = a.samples + ((size_t)t.seg * g.nodes + t.node) * g.m;
        const int32_t* pk = a.perm_k + t.slice;
        const int32_t* rk = a.rank_k + t.slice;
        for (int c00 = lane; c00 < nblk; c00 += 32 * UB) {
          int idx[UB];
#pragma unroll
          for (int u = 0; u < UB; ++u) {
            const int c0 = c00 + u * 32;
            idx[u] = -1;
            if (c0 < nblk) {
              const int which = c0 >= bcols;
              const int c = c0 - which * bcols;
              if (c < block_len(t.nk, g.b, which ? qb.beta : qa.beta)) idx[u] = pk[(size_t)(which ? qb.beta : qa.beta) * g.b + c];
            }
          }
#pragma unroll
          for (int u = 0; u < UB; ++u) {
            const int c0 = c00 + u * 32;
            if (c0 - lane < nblk) {                       // warp-uniform (nblk is a multiple of 32)
              const unsigned pad = __ballot_sync(0xffffffffu, idx[u] < 0);
              s_kidx[c0] = segrow_k + (idx[u] < 0 ? 0 : t.k0 + idx[u]);
              if (lane == 0) { s_mask[c0 >> 5] = pad; s_mask[MW + (c0 >> 5)] = pad; }
            }
          }
        }
        // Sampled columns: masked where the sample falls into the tile's own block (the factor
        // (1 - M^H) of Alg. 2 line 7).  The samples are an unordered multiset, so the masked ones
        // (for either query tile) are moved to the end of the sample part: only its last tile(s)
        // then carry mask bits, every other sampled tile takes the softmax warps' fast path.
        if (nblk < ncols) {
          for (int wd = (nblk >> 5) + lane; wd < (ncols >> 5); wd += 32) { s_mask[wd] = 0; s_mask[MW + wd] = 0; }
          __syncwarp();
          int nfront = 0, nback = 0;                      // unmasked samples placed from the front, masked ones from the back
          float* s_bias = reinterpret_cast<float*>(smem + C::kOffBias) + set * kMaxWeightedSamples;
          const float* swl = a.sample_wlog ? a.sample_wlog + ((size_t)t.seg * g.nodes + t.node) * g.m : nullptr;
          float bmax = -INFINITY;
          const unsigned lt_mask = (1u << lane) - 1u;
          for (int c00 = lane; c00 < ncols - nblk; c00 += 32 * UB) {
            int l[UB], blk[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
              const int c = c00 + u * 32;
              l[u] = c < g.m ? smp[c] : -1;
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) blk[u] = l[u] >= 0 ? rk[l[u]] / g.b : -1;
#pragma unroll
            for (int u = 0; u < UB; ++u) {
              const int c = c00 + u * 32;
              if (c - lane < ncols - nblk) {              // warp-uniform
                const bool valid = l[u] >= 0;
                const bool m0 = !valid || blk[u] == qa.beta;
                const bool m1 = !valid || (qb.valid && blk[u] == qb.beta);
                const unsigned bf = __ballot_sync(0xffffffffu, valid && !(m0 || m1));
                const unsigned bb = __ballot_sync(0xffffffffu, valid && (m0 || m1));
                int pos;
                if (!valid) pos = nblk + c;                                             // padding stays where it is (behind all samples)
                else if (!(m0 || m1)) pos = nblk + nfront + __popc(bf & lt_mask);
                else pos = nblk + g.m - 1 - (nback + __popc(bb & lt_mask));
                nfront += __popc(bf); nback += __popc(bb);
                s_kidx[pos] = segrow_k + (valid ? t.k0 + l[u] : 0);
                if (CAPPED && swl) {                      // weighted sampling: the column's own log2 weight travels with it
                  const float wl = valid ? swl[c] : 0.f;
                  s_bias[pos - nblk] = wl;
                  if (valid) bmax = fmaxf(bmax, wl);
                }
                if (m0) atomicOr(&s_mask[pos >> 5], 1u << (pos & 31));
                if (m1) atomicOr(&s_mask[MW + (pos >> 5)], 1u << (pos & 31));
              }
            }
          }
          if (CAPPED && swl) {
#pragma unroll
            for (int o = 16; o; o >>= 1) bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, o));
            if (lane == 0) reinterpret_cast<ItemDesc*>(smem + C::kOffDesc + set * C::kDescBytes)->t.bias_max = bmax;
          }
        }
      }
      if (lane == 0) HA_TACC(23, ttab);
      // query rows of both tiles: lane l owns rows 4l .. 4l+3
      int qr[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const QTile& q = i ? qb : qa;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int r = 4 * lane + k;
          qr[i][k] = -1;
          if (q.valid && r < q.nq) qr[i][k] = t.mode == 1 ? t.qnode0 + a.perm_q[t.slice + q.spos0 + r] : q.q0 + r;
        }
      }
#pragma unroll
      for (int i = 0; i < 2; ++i)
        *reinterpret_cast<int4*>(s_qrow + i * 128 + 4 * lane) = make_int4(qr[i][0], qr[i][1], qr[i][2], qr[i][3]);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tabfull(set));       // (release: the table writes of all lanes are ordered before it by the warp barrier)
      if (lane == 0) HA_TACC(10, ttab);
      // Sorted query rows are read once in the whole forward pass, so they come from HBM: ask for
      // them now (the softmax threads gather them a whole item later) so that they are found in L2.
      if (t.mode == 1) {
        const char* qbase = reinterpret_cast<const char*>(a.q) + (size_t)segrow * (D * 2);
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (qr[i][k] >= 0) {
#pragma unroll
              for (int ln = 0; ln < D * 2 / 128; ++ln)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(qbase + (size_t)qr[i][k] * (D * 2) + ln * 128));
            }
      }
      // ---- Q (the issuers must be done with the previous item's Q) ----------------------------
      HA_T0(tqf);
      if (it >= 1) {
        ok = mbar_wait<100, 17>(bar_qfree, (it - 1) & 1, s_abort, status);
        if (!ok) break;
      }
      if (lane == 0) HA_TACC(27, tqf);
      HA_T0(tqi);
      if (t.mode == 0) {
        // consecutive rows: one box per 64 columns and tile (rows past the tile's end are other
        // rows of the tensor or zeros: their results are never stored)
        if (lane == 0) {
          mbar_expect_tx(bar_q, (uint32_t)((qa.valid + qb.valid) * C::kQTile));
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (!(i ? qb.valid : qa.valid)) continue;
#pragma unroll
            for (int sl = 0; sl < D / 64; ++sl)
              tma_tile(ubase + C::kOffQ + i * C::kQTile + sl * (128 * 128), &maps.q, sl * 64, segrow + (i ? qb.q0 : qa.q0), bar_q);
          }
        }
        mbar_arrive(bar_q);
      } else {
        mbar_arrive(bar_q);                               // (the softmax threads gather these tiles)
      }
      if (lane == 0) { HA_TACC(25, ttab); HA_TACC(28, tqi); }
    }
    cp_async_commit();
    cp_async_wait_all();
    if (it > 0) mbar_drain(bar_q, (it - 1) & 1);
  } else {
    constexpr int CPR = D / 8;
    // ================= K / V streamer: key tiles of all items through the stage ring ====================
    // Tiles of consecutive rows: lane 0 issues one TMA box per 64 columns.  Gathered tiles: lane ->
    // column chunk cc and the row quads {4 (rq + k R) .. + 3}, R = 32 / CPR; the four row
    // coordinates of a quad come with one shared-memory load, and the swizzled destination of
    // every copy is the lane's base plus a compile-time offset (the swizzle phase (row & 7) of
    // row e of a quad is 4 (rq & 1) + e for every quad of the lane, R being even).
    bool ok = true;
    int gbase = 0;
    int it = 0;
    int k_armed = 0, v_armed = 0;                         // tiles whose K / V copies have been issued (all items)
    constexpr int R = 32 / CPR;                            // row quads covered by the warp per step
    constexpr int QUADS = (TK / 4) / R;                    // steps per tile
    const int cc = lane % CPR, rq = lane / CPR;
    uint32_t doff[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      doff[e] = (uint32_t)((cc >> 3) * (TK * 128) + (4 * rq + e) * 128 + (((cc & 7) ^ ((4 * rq + e) & 7)) << 4));
    const char* ksrc = reinterpret_cast<const char*>(a.k) + cc * 16;
    const char* vsrc = reinterpret_cast<const char*>(a.v) + cc * 16;
    for (; ok; ++it) {
      const int set = it & 1;
      const int* s_kidx = s_kidx_all + set * kMaxNodeKeys;
      ok = mbar_wait<100, 18>(bar_tabfull(set), (it >> 1) & 1, s_abort, status);
      if (!ok) break;
      const PairDesc t = reinterpret_cast<const ItemDesc*>(smem + C::kOffDesc + set * C::kDescBytes)->t;
      if (t.mode < 0) break;
      const int segrow = t.seg * g.nk;                      // (keys)
      for (int j = 0; j < t.ntiles && ok; ++j) {
        const int gj = gbase + j;
        const int s = gj % C::NS;
        const int use = gj / C::NS;
        int4 rows[QUADS];
        if (t.mode == 1) {
#pragma unroll
          for (int k = 0; k < QUADS; ++k) rows[k] = *reinterpret_cast<const int4*>(s_kidx + j * TK + 4 * (rq + k * R));
        }
        auto fill = [&](uint32_t stage, const CUtensorMap* map, const char* src, uint32_t bar) {
          if (t.mode == 0) {
            // (rows past the end of the key range are masked by the softmax warps)
            if (lane == 0) {
              mbar_expect_tx(bar, C::kTile);
#pragma unroll
              for (int sl = 0; sl < D / 64; ++sl) tma_tile(stage + sl * (TK * 128), map, sl * 64, segrow + t.k0 + j * TK, bar);
            }
            mbar_arrive(bar);
          } else {
#pragma unroll
            for (int k = 0; k < QUADS; ++k) {
              const uint32_t d = stage + k * (4 * R * 128);
              cp_async16(d + doff[0], src + (size_t)(uint32_t)rows[k].x * (D * 2));
              cp_async16(d + doff[1], src + (size_t)(uint32_t)rows[k].y * (D * 2));
              cp_async16(d + doff[2], src + (size_t)(uint32_t)rows[k].z * (D * 2));
              cp_async16(d + doff[3], src + (size_t)(uint32_t)rows[k].w * (D * 2));
            }
            cp_async_arrive_noinc(bar);
          }
        };
        HA_T0(tle);
        if (use > 0) {
          ok = mbar_wait<100, 10>(bar_kempty(0, s), (use - 1) & 1, s_abort, status);
          ok = ok && mbar_wait<100, 11>(bar_kempty(1, s), (use - 1) & 1, s_abort, status);
          if (!ok) break;
        }
        if (lane == 0) HA_TACC(11, tle);
        HA_T0(tgk);
        fill(ubase + C::kOffK + s * C::kTile, &maps.k, ksrc, bar_kfull(s));
        k_armed = gj + 1;
        if (lane == 0) HA_TACC(3, tgk);
        HA_T0(tle2);
        if (use > 0) {
          ok = mbar_wait<100, 12>(bar_vempty(0, s), (use - 1) & 1, s_abort, status);
          ok = ok && mbar_wait<100, 13>(bar_vempty(1, s), (use - 1) & 1, s_abort, status);
          if (!ok) break;
        }
        if (lane == 0) HA_TACC(11, tle2);
        HA_T0(tgv);
#ifdef HA_TEST_DROP_ARRIVAL
        {
          int drop = 0;
          if (lane == 0 && gj == 1) drop = atomicExch(&g_test_drop_armed, 0);
          if (__shfl_sync(0xffffffffu, drop, 0)) { v_armed = gj; continue; }     // nothing issued, nothing will arrive
        }
#endif
        fill(ubase + C::kOffV + s * C::kTile, &maps.v, vsrc, bar_vfull(s));
        v_armed = gj + 1;
        if (lane == 0) HA_TACC(1, tgv);
      }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tabfree(set));       // done reading this item's key rows
      gbase += t.ntiles;
    }
    // nothing may be in flight into shared memory when the CTA exits (trivially true unless it is giving up)
    cp_async_commit();
    cp_async_wait_all();
    for (int s = 0; s < C::NS; ++s) {
      if (k_armed > s) mbar_drain(bar_kfull(s), ((k_armed - 1 - s) / C::NS) & 1);   // phase of the last tile that used stage s
      if (v_armed > s) mbar_drain(bar_vfull(s), ((v_armed - 1 - s) / C::NS) & 1);
    }
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

#ifdef HA_TEST_DROP_ARRIVAL
extern "C" int hyperattn_test_arm_drop(int on) {
  return cudaMemcpyToSymbol(g_test_drop_armed, &on, sizeof(int)) == cudaSuccess ? 0 : -5;
}
#endif

#ifdef HA_TC_TIMING
extern "C" int hyperattn_debug_tc_timing(unsigned long long* host16, int reset) {
  if (cudaMemcpyFromSymbol(host16, g_tc_timing, sizeof(unsigned long long) * 48) != cudaSuccess) return -5;
  if (reset) { unsigned long long z[48] = {0}; cudaMemcpyToSymbol(g_tc_timing, z, sizeof(z)); }
  return 0;
}
#endif

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// the driver's tensor-map encoder, looked up through the runtime (no link against libcuda)
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace

// [rows x d] bf16, row-major; one box = 64 columns x box_rows rows (one slab of an operand tile).
// (Also used by the backward pass's launcher.)
bool encode_rows_map(CUtensorMap* m, const void* base, size_t rows, int d, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st) {
  if (a.total_pairs == 0) return cudaSuccess;
  const size_t rows = (size_t)a.g.G * a.g.n, rows_k = (size_t)a.g.G * a.g.nk;
  if (rows > 0x7fffffffull || rows_k > 0x7fffffffull) return cudaErrorInvalidValue;        // row coordinates are 32-bit
  TmaMaps maps;
  if (!encode_rows_map(&maps.q, a.q, rows, a.g.d, 128) || !encode_rows_map(&maps.k, a.k, rows_k, a.g.d, TK) ||
      !encode_rows_map(&maps.v, a.v, rows_k, a.g.d, TK)) return cudaErrorInvalidValue;
  auto go = [&](auto kernel, int smem_bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorUnknown;
    int grid = a.total_pairs < sms ? a.total_pairs : sms;     // persistent: one CTA per SM walks the item list
    kernel<<<grid, 384, smem_bytes, st>>>(a, maps, status);
    return cudaGetLastError();
  };
  if (a.capped || a.sample_wlog) {
    if (a.precise || (a.capped && a.sample_wlog)) return cudaErrorInvalidValue;
    if (a.g.d == 64) return go(attn_tc_kernel<64, false, false, true>, Cfg<64>::kTotal);
    if (!a.direct && !a.part_bf16) return go(attn_tc_kernel<128, true, false, true>, Cfg<128>::kTotal);
    return go(attn_tc_kernel<128, false, false, true>, Cfg<128>::kTotal);
  }
  if (a.precise) {
    if (a.g.d == 64) return go(attn_tc_kernel<64, false, true, false>, Cfg<64>::kTotal);
    if (!a.direct && !a.part_bf16) return go(attn_tc_kernel<128, true, true, false>, Cfg<128>::kTotal);
    return go(attn_tc_kernel<128, false, true, false>, Cfg<128>::kTotal);
  }
  if (a.g.d == 64) return go(attn_tc_kernel<64, false, false, false>, Cfg<64>::kTotal);
  if (!a.direct && !a.part_bf16) return go(attn_tc_kernel<128, true, false, false>, Cfg<128>::kTotal);
  return go(attn_tc_kernel<128, false, false, false>, Cfg<128>::kTotal);
}

}  // namespace hyperattn
