// Combining the partial results of the causal recursion (Alg. 4 line 5 carried through to
// the outputs): a row of the second half of a recursion node adds the estimated row sums
// D~_21 + D~_C22, so its output is the sum of the partial outputs weighted by their share of
// the total row sum.  Every row owns one exact-leaf partial and one partial per recursion
// level at which it sits in a second half.  HBM-bound: reads the partials once, writes
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

// LM: compile-time bound on the recursion depth; PB: bf16 partials and results (else fp32).
// A warp owns 32 consecutive rows.  First lane = row: the row's log-sum-exp values (its leaf partial and one partial
// per level at which it sits in a second half), its weights and where its partial rows are - once per row.  Then the
// data: LPR lanes per row, whole rows per warp instruction on every side, the weights and row offsets handed round by
// shuffles; KB row groups and all their levels are in flight together.  (One thread per 16 bytes of a row doing all
// of this on its own - the layout before - spent 385 instructions per thread, 56 % of the issue slots, and reached
// 60 % of the memory bandwidth.)
// (Occupancy matters more than loads in flight per thread: C3 0.416 ms with four resident CTAs of 64 registers,
// 0.52 ms with the compiler's 88; d = 128 does best with three and two row groups.)
template <int D, int LM, bool PB>
__global__ void __launch_bounds__(256, LM <= 8 ? (D == 64 ? 4 : 3) : 1) merge_kernel(MergeArgs a) {
  constexpr int ES = PB ? 2 : 4, RBY = D * ES;     // bytes per element and per row
  constexpr int LPR = RBY / 16 < 32 ? RBY / 16 : 32;   // lanes per row
  constexpr int CI = RBY / 16 / LPR;               // 16-byte chunks per lane and row (2 for fp32 rows of d = 128)
  constexpr int RPS = 32 / LPR;                    // rows per warp instruction
  constexpr int KB = (CI == 1 && LPR > 8) ? 2 : 1; // row groups in flight together (rows of 128 bytes do best one group at a time)
  constexpr int NE = 16 / ES;                      // entries per chunk
  constexpr int LG = LM <= 5 ? LM : 4;             // levels whose rows are in flight together
  const Geometry& g = a.g;
  const int seg = blockIdx.y;
  const int lane = threadIdx.x & 31;
  const int row0 = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32;
  if (row0 >= g.n) return;
  const int nr = min(32, g.n - row0);              // rows of this warp
  // ---- lane = row ---------------------------------------------------------------------------------------
  const int i = row0 + lane;
  const bool live = lane < nr;
  // a node of level `level` has s = leaf << (L - 1 - level) rows per half, so the row's place in every level follows
  // from its leaf number by shifts
  const int leaf_no = i / g.leaf;
  const int in_leaf = i - leaf_no * g.leaf;
  unsigned present = 0;
  uint32_t off[LM];                                // the row's partial row at a level, counted from the segment's first row of that level
  float w[LM];
  float wself = live ? __ldcs(a.part_lse + (size_t)seg * g.n + i) : 0.f;
  float mx = wself;
#pragma unroll
  for (int level = 0; level < LM; ++level) {
    w[level] = -INFINITY; off[level] = 0;
    const int sh = g.L - 1 - level;
    if (live && level < g.L && ((leaf_no >> sh) & 1)) {
      present |= 1u << level;
      off[level] = (uint32_t)(((size_t)(leaf_no >> (sh + 1)) << sh) * g.leaf + (size_t)(leaf_no & ((1 << sh) - 1)) * g.leaf + in_leaf);
      w[level] = __ldcs(a.part_lse + (size_t)g.G * g.n + ((size_t)level * g.G + seg) * g.nl + off[level]);
      mx = fmaxf(mx, w[level]);
    }
  }
  wself = __expf(wself - mx);
  float tot = wself;
#pragma unroll
  for (int level = 0; level < LM; ++level) { w[level] = __expf(w[level] - mx); tot += w[level]; }   // exp(-inf) = 0 for the absent ones
  const float inv = 1.f / tot;
  wself *= inv;
#pragma unroll
  for (int level = 0; level < LM; ++level) w[level] *= inv;
  if (live) a.lse[(size_t)seg * g.n + i] = mx + __logf(tot);
  const unsigned any_present = __reduce_or_sync(0xffffffffu, present);
  // ---- LPR lanes per row ----------------------------------------------------------------------------------
  const int crow = lane / LPR, cc = lane % LPR;
  const char* pself = reinterpret_cast<const char*>(a.part_o) + ((size_t)seg * g.n + row0) * RBY + cc * 16;
  auto unpack = [&](const uint4& v, float (&x)[NE]) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (PB) { x[2 * e] = __uint_as_float(u[e] << 16); x[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u); }
      else x[e] = __uint_as_float(u[e]);
    }
  };
  const int oes = (PB || a.out_fp32) ? ES : 2;     // bytes per entry of the results (fp32 partials may end as bf16 rows)
  char* pout = reinterpret_cast<char*>(a.out) + ((size_t)seg * g.n + row0) * (size_t)(D * oes);
#pragma unroll 1
  for (int sb = 0; sb * RPS < nr; sb += KB) {
#pragma unroll
    for (int ci = 0; ci < CI; ++ci) {
      uint4 xs[KB];
      float acc[KB][NE];
      int rl[KB];                                    // the row of the warp this lane works on
#pragma unroll
      for (int kk = 0; kk < KB; ++kk) {
        rl[kk] = (sb + kk) * RPS + crow;
        xs[kk] = rl[kk] < nr ? __ldcs(reinterpret_cast<const uint4*>(pself + (size_t)rl[kk] * RBY + ci * (LPR * 16))) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int l0 = 0; l0 < LM; l0 += LG) {
        if (l0 > 0 && ((any_present >> l0) & ((1u << LG) - 1u)) == 0) continue;
        uint4 x[KB][LG];
        float wl[KB][LG];
#pragma unroll
        for (int kk = 0; kk < KB; ++kk) {
          const unsigned pr = __shfl_sync(0xffffffffu, present, rl[kk] & 31);
#pragma unroll
          for (int lv = 0; lv < LG; ++lv) {
            const int level = l0 + lv;
            if (level >= LM || !((any_present >> level) & 1u)) continue;
            wl[kk][lv] = __shfl_sync(0xffffffffu, w[level], rl[kk] & 31);
            const uint32_t o = __shfl_sync(0xffffffffu, off[level], rl[kk] & 31);
            x[kk][lv] = make_uint4(0, 0, 0, 0);
            if (rl[kk] < nr && ((pr >> level) & 1u))
              x[kk][lv] = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.part_o)
                                 + ((size_t)g.G * g.n + ((size_t)level * g.G + seg) * g.nl + o) * RBY + cc * 16 + ci * (LPR * 16)));
          }
        }
        if (l0 == 0) {
#pragma unroll
          for (int kk = 0; kk < KB; ++kk) {
            const float ws = __shfl_sync(0xffffffffu, wself, rl[kk] & 31);
            float v[NE];
            unpack(xs[kk], v);
#pragma unroll
            for (int e = 0; e < NE; ++e) acc[kk][e] = ws * v[e];
          }
        }
#pragma unroll
        for (int kk = 0; kk < KB; ++kk) {
#pragma unroll
          for (int lv = 0; lv < LG; ++lv) {
            const int level = l0 + lv;
            if (level >= LM || !((any_present >> level) & 1u)) continue;
            float v[NE];
            unpack(x[kk][lv], v);
#pragma unroll
            for (int e = 0; e < NE; ++e) acc[kk][e] = fmaf(wl[kk][lv], v[e], acc[kk][e]);
          }
        }
      }
#pragma unroll
      for (int kk = 0; kk < KB; ++kk) {
        if (rl[kk] >= nr) continue;
        char* dst = pout + ((size_t)rl[kk] * D + (size_t)(ci * LPR + cc) * NE) * oes;
        if (PB) {
          uint32_t q[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 t2 = __floats2bfloat162_rn(acc[kk][2 * e], acc[kk][2 * e + 1]);
            q[e] = *reinterpret_cast<uint32_t*>(&t2);
          }
          __stcs(reinterpret_cast<uint4*>(dst), make_uint4(q[0], q[1], q[2], q[3]));
        } else if (a.out_fp32) {
          __stcs(reinterpret_cast<float4*>(dst), make_float4(acc[kk][0], acc[kk][1], acc[kk][2], acc[kk][3]));
        } else {
          __nv_bfloat162 t0 = __floats2bfloat162_rn(acc[kk][0], acc[kk][1]), t1 = __floats2bfloat162_rn(acc[kk][2], acc[kk][3]);
          __stcs(reinterpret_cast<uint2*>(dst), make_uint2(*reinterpret_cast<uint32_t*>(&t0), *reinterpret_cast<uint32_t*>(&t1)));
        }
      }
    }
  }
}

}  // namespace

cudaError_t launch_merge(const Geometry& g, const Workspace& ws, void* out, float* lse, int out_fp32,
                         cudaStream_t st) {
  MergeArgs a; a.part_o = ws.part_o; a.part_lse = ws.part_lse; a.out = out; a.lse = lse; a.g = g; a.out_fp32 = out_fp32;
  if (ws.part_bf16 && out_fp32) return cudaErrorInvalidValue;                   // bf16 partials are only kept for bf16 results
  const size_t warps = ((size_t)g.n + 31) / 32;                                 // a warp per 32 rows
  const dim3 blocks((unsigned)((warps + 7) / 8), (unsigned)g.G);
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
