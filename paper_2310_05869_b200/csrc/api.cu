// C ABI of the HyperAttention forward library: argument checks, workspace plan, stage
// sequencing.  Everything here runs on the host; all arithmetic of the method runs in the
// kernels of hash.cu, sort.cu, attn_*.cu and merge.cu.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <vector>

#include "../../include/hyperattn.h"
#include "attn_common.cuh"

namespace hyperattn {
cudaError_t launch_attention_mma(const AttnArgs& a, cudaStream_t st);
cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st);
cudaError_t launch_vnorm_sampling(const Geometry& g, const __nv_bfloat16* v, uint32_t* wq, unsigned long long* cum, int32_t* samples,
                                  float* wlog, uint64_t seed, cudaStream_t st);
cudaError_t launch_tau(const AttnArgs& at, const int32_t* tpos, float* ltau, cudaStream_t st);
cudaError_t launch_backward(const AttnArgs& a, const void* out, int out_fp32, const float* lse, const void* dout,
                            float* delta, float* dq, float* dk, float* dv, void* dq_final, int dq_mode, float scale, int* status, cudaStream_t st);
cudaError_t launch_to_bf16(const float* src, void* dst, size_t count, cudaStream_t st);

namespace {

constexpr int kVersion = 2;
constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// ---- geometry / validation ---------------------------------------------------------------
int build_geometry(const hyperattn_params& p, Geometry& g) {
  if (p.B <= 0 || p.H <= 0 || p.n <= 0 || p.block <= 0 || p.samples < 0 || p.n_k < 0) return HYPERATTN_INVALID_ARGUMENT;
  if (p.dtype != HYPERATTN_BF16 && p.dtype != HYPERATTN_FP32) return HYPERATTN_INVALID_ARGUMENT;
  if (p.out_dtype != HYPERATTN_BF16 && p.out_dtype != HYPERATTN_FP32) return HYPERATTN_INVALID_ARGUMENT;
  if (p.d != 64 && p.d != 128) return HYPERATTN_UNSUPPORTED_SHAPE;
  if (p.hash_bits < 1 || p.hash_bits > 8) return HYPERATTN_UNSUPPORTED_SHAPE;
  if ((long long)p.B * p.H > (1 << 20)) return HYPERATTN_UNSUPPORTED_SHAPE;
  if (p.n > (1 << 28) || p.n_k > (1 << 28)) return HYPERATTN_UNSUPPORTED_SHAPE;
  const int nk = p.n_k ? p.n_k : p.n;
  if (p.causal && nk != p.n) return HYPERATTN_UNSUPPORTED_SHAPE;       // the causal mask is defined for a square matrix
  std::memset(&g, 0, sizeof(g));
  g.seg0 = 0;
  g.G = p.B * p.H; g.n = p.n; g.nk = nk; g.npad = p.n; g.d = p.d; g.b = p.block; g.m = p.samples; g.r = p.hash_bits;
  g.bq = p.block;
  if (!p.causal) {
    g.causal = 0; g.L = 0; g.leaf = p.n; g.unit = p.n; g.unit_k = nk;
    g.nl = p.n > nk ? p.n : nk;
    if (p.block < nk) {
      g.levels = 1; g.nodes = 1; g.sorted = 1;
      g.bq = query_group(p.block, p.n, nk);
    }
  } else {
    if (p.n0 <= 0) return HYPERATTN_INVALID_ARGUMENT;
    g.causal = 1;
    // Alg. 4 halves the problem until a part is not longer than n0: L levels, 2^L leaves of
    // leaf = ceil(n / 2^L) rows.  The recursion cuts every part at half of its nominal length
    // leaf 2^k; when 2^L does not divide n the rows beyond n do not exist, so the last leaf and
    // the query side of a level's last node are short.
    int L = 0;
    while ((((long long)p.n + (1ll << L) - 1) >> L) > p.n0 && L <= kMaxLevels) ++L;
    if (L > kMaxLevels) return HYPERATTN_UNSUPPORTED_SHAPE;
    g.L = L;
    g.leaf = (int)(((long long)p.n + (1ll << L) - 1) >> L);
    if (((long long)g.leaf << L) > (1ll << 29)) return HYPERATTN_UNSUPPORTED_SHAPE;
    g.npad = g.leaf << L;
    g.unit = g.leaf; g.unit_k = g.leaf;
    g.nl = p.n;
    if (L) {
      g.levels = L; g.nl = g.npad / 2; g.nodes = (1 << L) - 1;
      for (int l = 0; l < L; ++l) {
        const int s = g.npad >> (l + 1);
        if (p.block < s) g.sorted = 1;
      }
    }
  }
  if (g.sorted) {
    const int bpad = (g.b + 127) / 128 * 128, mpad = (g.m + 127) / 128 * 128;
    if (2 * bpad + mpad > kMaxNodeKeys) return HYPERATTN_UNSUPPORTED_SHAPE;
  }
  g.chunks_per_unit = (g.unit + kSortChunk - 1) / kSortChunk;
  g.chunks_per_seg = (g.npad / g.unit) * g.chunks_per_unit;
  g.chunks_per_unit_k = (g.unit_k + kSortChunk - 1) / kSortChunk;
  g.chunks_per_seg_k = g.causal ? g.chunks_per_seg : g.chunks_per_unit_k;
  return HYPERATTN_OK;
}

struct Plan {
  size_t q16, k16, v16, q16lo, k16lo, ids, hist, offs, perm_q, perm_k, rank_k, samples, tpos, ltau, vwq, vcum, swlog, wnodes, sched, part_o, part_lse, total;
  size_t delta, gacc;   // backward only: <dO, O> per row; fp32 gradient accumulators (bf16 gradients only)
};

// backward: 0 forward plan; 1 backward with fp32 gradients (accumulated in place); 2 backward with bf16 gradients
Plan make_plan(const Geometry& g, int is_fp32, int backward = 0, bool capped = false, bool vnorm = false, bool part_bf16 = false) {
  Plan pl;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  const size_t tensor16 = (size_t)g.G * g.n * g.d * 2, tensor16k = (size_t)g.G * g.nk * g.d * 2;
  pl.q16 = take(is_fp32 ? tensor16 : 0);
  pl.k16 = take(is_fp32 ? tensor16k : 0);
  pl.v16 = take(is_fp32 ? tensor16k : 0);
  pl.q16lo = take(is_fp32 ? tensor16 : 0);
  pl.k16lo = take(is_fp32 ? tensor16k : 0);
  const size_t lvl_rows = (size_t)g.levels * g.G * g.nl;
  const size_t id_sets = g.node_dirs ? g.levels : 1;     // directions of the nodes' own: ids and histograms once per level
  pl.ids = take(g.sorted ? id_sets * g.G * ((size_t)g.n + g.nk) : 0);
  pl.hist = take(g.sorted ? id_sets * g.G * (g.chunks_per_seg + g.chunks_per_seg_k) * kBuckets * 4 : 0);
  pl.wnodes = take(g.node_dirs ? (size_t)g.nodes * g.d * g.r * 4 : 0);
  const size_t chunks_per_level = g.sorted ? (size_t)side_cpl(g, 0) + side_cpl(g, 1) : 0;
  pl.offs = take((size_t)g.levels * g.G * chunks_per_level * kBuckets * 4);
  pl.perm_q = take(g.sorted ? lvl_rows * 4 : 0);
  pl.perm_k = take(g.sorted ? lvl_rows * 4 : 0);
  pl.rank_k = take(g.sorted ? lvl_rows * 4 : 0);
  pl.samples = take((size_t)g.G * g.nodes * g.m * 4);
  pl.sched = take(256);
  pl.tpos = take(capped ? (size_t)g.G * g.nodes * g.m * 4 : 0);
  pl.ltau = take(capped ? (size_t)g.G * g.nodes * 4 : 0);
  pl.vwq = take(vnorm ? (size_t)g.G * g.nk * 4 : 0);
  pl.vcum = take(vnorm ? (size_t)g.G * ((size_t)g.nk + 1) * 8 : 0);
  pl.swlog = take(vnorm ? (size_t)g.G * g.nodes * g.m * 4 : 0);
  const size_t part_rows = (g.L && !backward) ? (size_t)g.G * g.n + lvl_rows : 0;
  pl.part_o = take(part_rows * g.d * (part_bf16 ? 2 : 4));
  pl.part_lse = take(part_rows * 4);
  pl.delta = take(backward ? (size_t)g.G * g.n * 4 : 0);
  pl.gacc = take(backward == 2 ? (size_t)3 * g.G * g.n * g.d * 4 : 0);
  pl.total = off + kAlign;
  return pl;
}

// ---- direction matrix (Def. 1): Philox + Box-Muller in fp64, rounded once to fp32 -------------
// node: 0 for the shared set; v for the directions of recursion node v's own (counter word 2)
void make_directions(int d, int r, uint64_t seed, float* w, uint32_t node = 0) {
  const int total = d * r, calls = (total + 3) / 4;
  const double two_pi = 6.283185307179586476925286766559;
  for (int c = 0; c < calls; ++c) {
    const Philox4 x = philox4x32_10((uint32_t)c, 0u, node, kDomainDirections, (uint32_t)seed, (uint32_t)(seed >> 32));
    double u[4], z[4];
    for (int i = 0; i < 4; ++i) u[i] = ((double)x.x[i] + 0.5) * (1.0 / 4294967296.0);
    for (int a = 0; a < 4; a += 2) {
      const double rho = std::sqrt(-2.0 * std::log(u[a])), ang = two_pi * u[a + 1];
      z[a] = rho * std::cos(ang);
      z[a + 1] = rho * std::sin(ang);
    }
    for (int i = 0; i < 4; ++i)
      if (4 * c + i < total) w[4 * c + i] = (float)z[i];
  }
}

// ---- per-process state ---------------------------------------------------------------------
constexpr int kHostChunks = 16;          // the host-buffer entry point pipelines copies and compute over this many groups of segments
struct DeviceState {
  void* ws = nullptr; size_t ws_bytes = 0;
  void* host_stage = nullptr; size_t host_stage_bytes = 0;   // device staging for the host-buffer entry
  int* status = nullptr;
  // host-buffer entry point: one stream per copy direction, events that order them with the caller's stream
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_end = nullptr, ev_in[kHostChunks] = {}, ev_done[kHostChunks] = {};
};
struct StageEvents { cudaEvent_t beg, end; int stage; int launches; };

std::mutex g_mu;
std::map<int, DeviceState> g_dev;
bool g_profile = false;
unsigned g_profile_mask = ~0u;          // stages that are timed while profiling is on
std::vector<StageEvents> g_events;
std::vector<cudaEvent_t> g_event_pool;
int g_profile_calls = 0;
struct { int d = 0, r = 0; uint64_t seed = 0; bool valid = false; float w[128 * 8]; } g_wcache;
// directions of the recursion nodes' own, [nodes, d, r]; kept on the host (it is copied to the device by every call that
// uses it, possibly from inside a captured graph, so the buffer only ever grows and is never freed before release)
struct { int d = 0, r = 0, nodes = 0; uint64_t seed = 0; std::vector<float> w; } g_wnodes;
constexpr int kMaxNodesOwnDirections = 4095;

cudaEvent_t take_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct StageScope {
  cudaStream_t st; int stage; int launches; bool on; cudaEvent_t beg = nullptr;
  StageScope(cudaStream_t s, int stage_, int launches_) : st(s), stage(stage_), launches(launches_), on(g_profile && launches_ > 0 && ((g_profile_mask >> stage_) & 1u)) {
    if (on) { beg = take_event(); cudaEventRecord(beg, st); }
  }
  ~StageScope() {
    if (on) { cudaEvent_t end = take_event(); cudaEventRecord(end, st); g_events.push_back({beg, end, stage, launches}); }
  }
};

int check_ptrs(const hyperattn_params& p) {
  if (!p.q || !p.k || !p.v || !p.out || !p.lse) return HYPERATTN_INVALID_ARGUMENT;
  const void* ptrs[5] = {p.q, p.k, p.v, p.out, p.lse};
  for (const void* x : ptrs)
    if (reinterpret_cast<uintptr_t>(x) & 15) return HYPERATTN_MISALIGNED;
  if (p.out == p.q || p.out == p.k || p.out == p.v || (void*)p.lse == p.out) return HYPERATTN_MISALIGNED;
  if (p.workspace && (reinterpret_cast<uintptr_t>(p.workspace) & 15)) return HYPERATTN_MISALIGNED;
  return HYPERATTN_OK;
}

// seg0: index of the call's first segment in the caller's whole tensor (not 0 when a caller's batch is
// processed in several calls: the samples of a segment depend on its index).  bw: run the backward
// pass instead (p->out and p->lse are then the forward pass's results, read only).
int forward_impl(const hyperattn_params& p, int seg0 = 0, const hyperattn_grads* bw = nullptr) {
  Geometry g;
  int rc = build_geometry(p, g);
  if (rc) return rc;
  g.seg0 = seg0;
  rc = check_ptrs(p);
  if (rc) return rc;
  // directions of every recursion node's own: only causal calls with sorted levels have more than one node
  g.node_dirs = p.node_directions != 0 && g.causal && g.L > 0 && g.sorted;
  if (g.node_dirs && (g.nodes > kMaxNodesOwnDirections || bw)) return HYPERATTN_UNSUPPORTED_SHAPE;
  const int is_fp32 = p.dtype == HYPERATTN_FP32;
  const int out_fp32 = p.out_dtype == HYPERATTN_FP32;
  if (bw) {
    if (is_fp32) return HYPERATTN_UNSUPPORTED_SHAPE;                 // the backward pass takes bf16 inputs
    if (g.nk != g.n || g.npad != g.n) return HYPERATTN_UNSUPPORTED_SHAPE;   // equal sides and causal lengths that 2^L divides only
    if (!bw->dout || !bw->dq || !bw->dk || !bw->dv) return HYPERATTN_INVALID_ARGUMENT;
    if (bw->grad_dtype != HYPERATTN_BF16 && bw->grad_dtype != HYPERATTN_FP32) return HYPERATTN_INVALID_ARGUMENT;
    for (const void* x : {bw->dout, (const void*)bw->dq, (const void*)bw->dk, (const void*)bw->dv})
      if (reinterpret_cast<uintptr_t>(x) & 15) return HYPERATTN_MISALIGNED;
  }
  // Alg. 2 with its caps: sorted nodes with samples only (elsewhere there is nothing to cap)
  const bool capped = p.capped != 0 && g.sorted && g.m > 0;
  if (p.capped != 0) {
    if (!(p.cap_scale > 0.f) || !(p.kappa > 0.f)) return HYPERATTN_INVALID_ARGUMENT;
    if (is_fp32 || bw || p.precise) return HYPERATTN_UNSUPPORTED_SHAPE;     // bf16 forward with single bf16 weights only
  }
  if (p.precise && is_fp32) return HYPERATTN_UNSUPPORTED_SHAPE;
  // sampled columns by squared row norms of V (Lemma 2) instead of uniformly (Sec. 4)
  if (p.sampling != HYPERATTN_SAMPLE_UNIFORM && p.sampling != HYPERATTN_SAMPLE_VALUE_NORMS) return HYPERATTN_INVALID_ARGUMENT;
  const bool vnorm = p.sampling == HYPERATTN_SAMPLE_VALUE_NORMS && g.sorted && g.m > 0;
  if (p.sampling == HYPERATTN_SAMPLE_VALUE_NORMS) {
    if (is_fp32 || bw || p.precise || p.capped) return HYPERATTN_UNSUPPORTED_SHAPE;
    if (g.m > kMaxWeightedSamples) return HYPERATTN_UNSUPPORTED_SHAPE;
  }
  // partial results of the causal recursion travel in the type of the final output (bf16 inputs only)
  const bool part_bf16 = !is_fp32 && !out_fp32 && g.L > 0;
  const Plan pl = make_plan(g, is_fp32, bw ? (bw->grad_dtype == HYPERATTN_FP32 ? 1 : 2) : 0, capped, vnorm, part_bf16);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState& ds = g_dev[dev];
  // While the stream is being captured into a graph nothing may be allocated or synchronised: the status word
  // and (without a caller's workspace) a large enough private workspace must exist already.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
  const bool capturing = cap != cudaStreamCaptureStatusNone;
  if (!ds.status) {
    if (capturing) return HYPERATTN_WORKSPACE_TOO_SMALL;
    if (cudaMalloc(&ds.status, 256) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
    if (cudaMemset(ds.status, 0, 256) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  }
  char* base = nullptr;
  if (p.workspace) {
    if (p.workspace_bytes < pl.total) return HYPERATTN_WORKSPACE_TOO_SMALL;
    base = reinterpret_cast<char*>(p.workspace);
  } else {
    if (ds.ws_bytes < pl.total && capturing) return HYPERATTN_WORKSPACE_TOO_SMALL;
    if (ds.ws_bytes < pl.total) {
      cudaDeviceSynchronize();
      if (ds.ws) cudaFree(ds.ws);
      ds.ws = nullptr; ds.ws_bytes = 0;
      if (cudaMalloc(&ds.ws, pl.total) != cudaSuccess) { cudaGetLastError(); return HYPERATTN_CUDA_ERROR; }
      ds.ws_bytes = pl.total;
    }
    base = reinterpret_cast<char*>(ds.ws);
  }
  base = reinterpret_cast<char*>(align_up(reinterpret_cast<uintptr_t>(base)));

  Workspace ws;
  ws.q16 = reinterpret_cast<__nv_bfloat16*>(base + pl.q16);
  ws.k16 = reinterpret_cast<__nv_bfloat16*>(base + pl.k16);
  ws.v16 = reinterpret_cast<__nv_bfloat16*>(base + pl.v16);
  ws.q16lo = reinterpret_cast<__nv_bfloat16*>(base + pl.q16lo);
  ws.k16lo = reinterpret_cast<__nv_bfloat16*>(base + pl.k16lo);
  ws.ids = reinterpret_cast<uint8_t*>(base + pl.ids);
  ws.hist = reinterpret_cast<uint32_t*>(base + pl.hist);
  ws.offs = reinterpret_cast<uint32_t*>(base + pl.offs);
  ws.perm_q = reinterpret_cast<int32_t*>(base + pl.perm_q);
  ws.perm_k = reinterpret_cast<int32_t*>(base + pl.perm_k);
  ws.rank_k = reinterpret_cast<int32_t*>(base + pl.rank_k);
  ws.samples = reinterpret_cast<int32_t*>(base + pl.samples);
  ws.tpos = capped ? reinterpret_cast<int32_t*>(base + pl.tpos) : nullptr;
  ws.ltau = capped ? reinterpret_cast<float*>(base + pl.ltau) : nullptr;
  ws.part_o = base + pl.part_o;
  ws.part_bf16 = part_bf16;
  ws.part_lse = reinterpret_cast<float*>(base + pl.part_lse);
  ws.status = ds.status;

  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.f / std::sqrt((float)p.d);
  const hyperattn_debug* dbg = p.debug;
  if (g_profile) ++g_profile_calls;
  cudaError_t e = cudaSuccess;
#define HA_CHECK(x) do { e = (x); if (e != cudaSuccess) { std::fprintf(stderr, "hyperattn: %s failed: %s\n", #x, cudaGetErrorString(e)); return HYPERATTN_CUDA_ERROR; } } while (0)

  const __nv_bfloat16 *q16 = reinterpret_cast<const __nv_bfloat16*>(p.q), *k16 = reinterpret_cast<const __nv_bfloat16*>(p.k),
                      *v16 = reinterpret_cast<const __nv_bfloat16*>(p.v);
  if (is_fp32) {
    StageScope sc(st, HYPERATTN_STAGE_CONVERT, 3);
    const size_t cnt = (size_t)g.G * g.n * g.d, cnt_k = (size_t)g.G * g.nk * g.d;
    HA_CHECK(launch_convert(reinterpret_cast<const float*>(p.q), ws.q16, ws.q16lo, cnt, st));
    HA_CHECK(launch_convert(reinterpret_cast<const float*>(p.k), ws.k16, ws.k16lo, cnt_k, st));
    HA_CHECK(launch_convert(reinterpret_cast<const float*>(p.v), ws.v16, nullptr, cnt_k, st));
    q16 = ws.q16; k16 = ws.k16; v16 = ws.v16;
  }
  if (g.sorted) {
    if (!g_wcache.valid || g_wcache.d != g.d || g_wcache.r != g.r || g_wcache.seed != p.seed) {
      make_directions(g.d, g.r, p.seed, g_wcache.w);
      g_wcache.d = g.d; g_wcache.r = g.r; g_wcache.seed = p.seed; g_wcache.valid = true;
    }
    const float* w_nodes = nullptr;
    if (g.node_dirs) {
      const size_t per = (size_t)g.d * g.r;
      if (g_wnodes.d != g.d || g_wnodes.r != g.r || g_wnodes.seed != p.seed || g_wnodes.nodes < g.nodes) {
        if (g_wnodes.w.size() < per * kMaxNodesOwnDirections) g_wnodes.w.resize(per * kMaxNodesOwnDirections);   // once: the address stays
        for (int v = 0; v < g.nodes; ++v) make_directions(g.d, g.r, p.seed, g_wnodes.w.data() + v * per, (uint32_t)v);
        g_wnodes.d = g.d; g_wnodes.r = g.r; g_wnodes.seed = p.seed; g_wnodes.nodes = g.nodes;
      }
      HA_CHECK(cudaMemcpyAsync(base + pl.wnodes, g_wnodes.w.data(), per * g.nodes * 4, cudaMemcpyHostToDevice, st));
      w_nodes = reinterpret_cast<const float*>(base + pl.wnodes);
    }
    {
      StageScope sc(st, HYPERATTN_STAGE_HASH, 1);
      HA_CHECK(launch_hash(g, p.q, p.k, is_fp32, g_wcache.w, ws, dbg ? dbg->near_zero_bits : nullptr, st, 3, w_nodes));
    }
    {
      // (the samples of Alg. 2 line 4 are drawn by extra blocks of this launch)
      StageScope sc(st, HYPERATTN_STAGE_SORT_SCAN, 1);
      HA_CHECK(launch_sort_scan(g, ws, !vnorm, p.seed, st));
    }
    if (vnorm) {
      StageScope sc(st, HYPERATTN_STAGE_SAMPLE, 3);
      HA_CHECK(launch_vnorm_sampling(g, v16, reinterpret_cast<uint32_t*>(base + pl.vwq), reinterpret_cast<unsigned long long*>(base + pl.vcum),
                                     ws.samples, reinterpret_cast<float*>(base + pl.swlog), p.seed, st));
      if (dbg && dbg->sample_log2w)
        HA_CHECK(cudaMemcpyAsync(dbg->sample_log2w, base + pl.swlog, (size_t)g.G * g.nodes * g.m * 4, cudaMemcpyDeviceToDevice, st));
    }
    {
      StageScope sc(st, HYPERATTN_STAGE_SORT_SCATTER, 1);
      HA_CHECK(launch_sort_scatter(g, ws, st));
    }
    if (dbg) {
      const size_t lvl_bytes = (size_t)g.levels * g.G * g.nl * 4;
      // (directions of the nodes' own: one set of ids per level, [LV, G, n] each)
      const int sets = g.node_dirs ? g.levels : 1;
      for (int l = 0; l < sets; ++l) {
        const uint8_t* src = ws.ids + l * ids_level_stride(g);
        if (dbg->q_ids) HA_CHECK(cudaMemcpyAsync(dbg->q_ids + (size_t)l * g.G * g.n, src, (size_t)g.G * g.n, cudaMemcpyDeviceToDevice, st));
        if (dbg->k_ids) HA_CHECK(cudaMemcpyAsync(dbg->k_ids + (size_t)l * g.G * g.nk, src + (size_t)g.G * g.n, (size_t)g.G * g.nk, cudaMemcpyDeviceToDevice, st));
      }
      if (dbg->perm_q) HA_CHECK(cudaMemcpyAsync(dbg->perm_q, ws.perm_q, lvl_bytes, cudaMemcpyDeviceToDevice, st));
      if (dbg->perm_k) HA_CHECK(cudaMemcpyAsync(dbg->perm_k, ws.perm_k, lvl_bytes, cudaMemcpyDeviceToDevice, st));
      if (dbg->rank_k) HA_CHECK(cudaMemcpyAsync(dbg->rank_k, ws.rank_k, lvl_bytes, cudaMemcpyDeviceToDevice, st));
      if (dbg->samples && g.m > 0)
        HA_CHECK(cudaMemcpyAsync(dbg->samples, ws.samples, (size_t)g.G * g.nodes * g.m * 4, cudaMemcpyDeviceToDevice, st));
    }
  }

  // ---- attention tiles: one launch over leaves and all recursion levels -------------------
  AttnArgs a;
  std::memset(&a, 0, sizeof(a));
  a.q = q16; a.k = k16; a.v = v16; a.g = g;
  if (is_fp32) { a.q_lo = ws.q16lo; a.k_lo = ws.k16lo; }
  a.scale_log2 = scale * 1.4426950408889634f;
  a.perm_q = ws.perm_q; a.perm_k = ws.perm_k; a.rank_k = ws.rank_k; a.samples = ws.samples;
  a.part_o = ws.part_o; a.part_lse = ws.part_lse; a.part_bf16 = part_bf16; a.out = p.out; a.lse = p.lse;
  a.out_fp32 = out_fp32;
  a.precise = p.precise != 0;
  a.capped = capped;
  a.cap_scale = p.cap_scale; a.log2_kappa = capped ? std::log2(p.kappa) : 0.f; a.ltau = ws.ltau;
  a.sample_wlog = vnorm ? reinterpret_cast<const float*>(base + pl.swlog) : nullptr;
  a.direct = g.L == 0;
  a.dense_causal = g.causal;
  a.tiles_per_block = (g.bq + kTileQ - 1) / kTileQ;
  const bool has_leaves = g.causal || !g.sorted;
  if (has_leaves) {
    a.tiles_per_leaf = (g.leaf + kTileQ - 1) / kTileQ;
    a.leaves_per_seg = g.npad / g.leaf;
    a.n_leaf_tiles = g.G * a.leaves_per_seg * a.tiles_per_leaf;
    a.pairs_per_leaf = (a.tiles_per_leaf + 1) / 2;
    a.n_leaf_pairs = g.G * a.leaves_per_seg * a.pairs_per_leaf;
  }
  long long tiles = a.n_leaf_tiles, pairs = a.n_leaf_pairs;
  for (int l = 0; l < g.levels; ++l) {
    int s, q0, k0;
    node_rows(g, l, 0, s, q0, k0);
    const int nodes_lvl = g.causal ? (1 << l) : 1;
    a.level_start[l] = (int)tiles;
    a.level_sorted[l] = g.b < s;
    const long long per_node = a.level_sorted[l] ? (long long)node_blocks(s, g.b) * a.tiles_per_block : ((g.causal ? s : g.n) + kTileQ - 1) / kTileQ;
    tiles += per_node * nodes_lvl * g.G;
    if (tiles > 0x7fffffffLL) return HYPERATTN_UNSUPPORTED_SHAPE;
    a.level_pair_start[l] = (int)pairs;
    // two query tiles share a CTA when they share their block's keys (even tiles per block),
    // or when a block is a single tile; other block sizes run one tile per CTA (a pair that
    // straddles two larger blocks would make each tile's issuer skip more key tiles of the
    // other's block than the stage ring holds, which the ring's release order does not allow)
    // (a single query tile per group only pairs up when the groups' key blocks are short as well: with fewer
    // queries than keys a group of at most 128 queries can face a key block of many tiles)
    a.level_paired[l] = !a.level_sorted[l] || a.tiles_per_block % 2 == 0 || (a.tiles_per_block == 1 && g.b <= kTileQ);
    pairs += (a.level_paired[l] ? (per_node + 1) / 2 : per_node) * nodes_lvl * g.G;
  }
  a.level_start[g.levels] = (int)tiles;
  a.total_tiles = (int)tiles;
  a.level_pair_start[g.levels] = (int)pairs;
  a.total_pairs = (int)pairs;
  if (bw) {
    const size_t elems = (size_t)g.G * g.n * g.d;
    const bool g32 = bw->grad_dtype == HYPERATTN_FP32;
    float* acc = reinterpret_cast<float*>(base + pl.gacc);
    float* dq = g32 ? reinterpret_cast<float*>(bw->dq) : acc;
    float* dk = g32 ? reinterpret_cast<float*>(bw->dk) : acc + elems;
    float* dv = g32 ? reinterpret_cast<float*>(bw->dv) : acc + 2 * elems;
    StageScope sc(st, HYPERATTN_STAGE_BACKWARD, 2 + (g32 ? 0 : 3));
    // without the causal recursion every query row belongs to one tile: the kernel writes dQ in its final type
    const int dq_mode = a.direct ? (g32 ? 1 : 2) : 0;
    if (!dq_mode) HA_CHECK(cudaMemsetAsync(dq, 0, elems * 4, st));
    HA_CHECK(cudaMemsetAsync(dk, 0, elems * 4, st));
    HA_CHECK(cudaMemsetAsync(dv, 0, elems * 4, st));
    HA_CHECK(launch_backward(a, p.out, out_fp32, p.lse, bw->dout, reinterpret_cast<float*>(base + pl.delta), dq, dk, dv, bw->dq, dq_mode, scale, ws.status, st));
    if (!g32) {
      if (!dq_mode) HA_CHECK(launch_to_bf16(dq, bw->dq, elems, st));
      HA_CHECK(launch_to_bf16(dk, bw->dk, elems, st));
      HA_CHECK(launch_to_bf16(dv, bw->dv, elems, st));
    }
    return HYPERATTN_OK;
  }
  if (capped) {
    // Alg. 2 line 3: the largest unmasked row sum among the probe rows of every node
    StageScope sc(st, HYPERATTN_STAGE_ATTENTION, 1);
    HA_CHECK(launch_tau(a, ws.tpos, ws.ltau, st));
    if (dbg && dbg->row_subset) HA_CHECK(cudaMemcpyAsync(dbg->row_subset, ws.tpos, (size_t)g.G * g.nodes * g.m * 4, cudaMemcpyDeviceToDevice, st));
    if (dbg && dbg->log2_tau) HA_CHECK(cudaMemcpyAsync(dbg->log2_tau, ws.ltau, (size_t)g.G * g.nodes * 4, cudaMemcpyDeviceToDevice, st));
  }
  {
    StageScope sc(st, HYPERATTN_STAGE_ATTENTION, 1);
    // bf16 inputs: tcgen05 path; fp32 inputs: split-bf16 logits on the warp-level MMA path
    if (is_fp32) HA_CHECK(launch_attention_mma(a, st));
    else {
      a.sched = reinterpret_cast<int*>(base + pl.sched);
      HA_CHECK(cudaMemsetAsync(a.sched, 0, 4, st));
      HA_CHECK(launch_attention_tc(a, ws.status, st));
    }
  }
  if (g.L) {
    StageScope sc(st, HYPERATTN_STAGE_MERGE, 1);
    HA_CHECK(launch_merge(g, ws, p.out, p.lse, out_fp32, st));
  }
#undef HA_CHECK
  return HYPERATTN_OK;
}

}  // namespace
}  // namespace hyperattn

using namespace hyperattn;

extern "C" {

int hyperattn_forward_ex(const hyperattn_params* p) {
  if (!p) return HYPERATTN_INVALID_ARGUMENT;
  return forward_impl(*p);
}

int hyperattn_backward(const hyperattn_params* p, const hyperattn_grads* grads) {
  if (!p || !grads) return HYPERATTN_INVALID_ARGUMENT;
  return forward_impl(*p, 0, grads);
}

int hyperattn_backward_workspace_bytes(const hyperattn_params* p, int grad_dtype, size_t* bytes) {
  if (!p || !bytes) return HYPERATTN_INVALID_ARGUMENT;
  Geometry g;
  const int rc = build_geometry(*p, g);
  if (rc) return rc;
  *bytes = make_plan(g, 0, grad_dtype == HYPERATTN_FP32 ? 1 : 2).total;
  return HYPERATTN_OK;
}

int hyperattn_forward(const void* q, const void* k, const void* v, void* out, float* lse, int B, int H, int n,
                      int d, int block, int samples, int hash_bits, int causal, int n0, uint64_t seed,
                      void* stream) {
  hyperattn_params p;
  std::memset(&p, 0, sizeof(p));
  p.q = q; p.k = k; p.v = v; p.out = out; p.lse = lse;
  p.B = B; p.H = H; p.n = n; p.d = d; p.block = block; p.samples = samples; p.hash_bits = hash_bits;
  p.causal = causal; p.n0 = n0; p.seed = seed;
  p.dtype = HYPERATTN_BF16; p.out_dtype = HYPERATTN_BF16; p.softmax_scale = 0.f;
  p.stream = stream;
  return forward_impl(p);
}

int hyperattn_forward_host(const hyperattn_params* hp) {
  if (!hp) return HYPERATTN_INVALID_ARGUMENT;
  if (!hp->q || !hp->k || !hp->v || !hp->out || !hp->lse) return HYPERATTN_INVALID_ARGUMENT;
  Geometry g;
  int rc = build_geometry(*hp, g);
  if (rc) return rc;
  const size_t es = hp->dtype == HYPERATTN_FP32 ? 4 : 2, eo = hp->out_dtype == HYPERATTN_FP32 ? 4 : 2;
  const size_t elems = (size_t)g.G * g.n * g.d, elems_k = (size_t)g.G * g.nk * g.d;
  const size_t in_b = align_up(elems * es), in_bk = align_up(elems_k * es), out_b = align_up(elems * eo), lse_b = align_up((size_t)g.G * g.n * 4);
  const size_t need = in_b + 2 * in_bk + out_b + lse_b;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  char* stage = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState& ds = g_dev[dev];
    if (ds.host_stage_bytes < need) {
      cudaDeviceSynchronize();
      if (ds.host_stage) cudaFree(ds.host_stage);
      ds.host_stage = nullptr; ds.host_stage_bytes = 0;
      if (cudaMalloc(&ds.host_stage, need) != cudaSuccess) { cudaGetLastError(); return HYPERATTN_CUDA_ERROR; }
      ds.host_stage_bytes = need;
    }
    stage = reinterpret_cast<char*>(ds.host_stage);
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(hp->stream);
  char* dq = stage; char* dk = stage + in_b; char* dv = stage + in_b + in_bk;
  char* dout = stage + in_b + 2 * in_bk; char* dlse = dout + out_b;
  // Segments are independent, so the batch goes through in groups: the copy of group c + 1 to the
  // device and the copy of group c - 1 back run (on streams of their own, PCIe being full duplex)
  // while group c is computed on the caller's stream.  With debug outputs requested, one group.
  DeviceState* dsp;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    dsp = &g_dev[dev];
    if (!dsp->copy_in) {
      bool good = cudaStreamCreateWithFlags(&dsp->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&dsp->copy_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&dsp->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&dsp->ev_end, cudaEventDisableTiming) == cudaSuccess;
      for (int c = 0; c < kHostChunks && good; ++c)
        good = cudaEventCreateWithFlags(&dsp->ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&dsp->ev_done[c], cudaEventDisableTiming) == cudaSuccess;
      if (!good) { dsp->copy_in = nullptr; return HYPERATTN_CUDA_ERROR; }
    }
  }
  DeviceState& ds = *dsp;
  const int nchunks = hp->debug ? 1 : (g.G < kHostChunks ? g.G : kHostChunks);
  const int per = (g.G + nchunks - 1) / nchunks;
  const size_t seg_in = (size_t)g.n * g.d * es, seg_ink = (size_t)g.nk * g.d * es, seg_out = (size_t)g.n * g.d * eo, seg_lse = (size_t)g.n * 4;
#define HA_HOST(x) do { if ((x) != cudaSuccess) { std::fprintf(stderr, "hyperattn: %s failed\n", #x); return HYPERATTN_CUDA_ERROR; } } while (0)
  // the staging buffers may still be in use by work queued earlier on the caller's stream
  HA_HOST(cudaEventRecord(ds.ev_start, st));
  HA_HOST(cudaStreamWaitEvent(ds.copy_in, ds.ev_start, 0));
  HA_HOST(cudaStreamWaitEvent(ds.copy_out, ds.ev_start, 0));
  for (int c = 0, s0 = 0; s0 < g.G; ++c, s0 += per) {
    const int ns = (g.G - s0) < per ? (g.G - s0) : per;
    const size_t oi = (size_t)s0 * seg_in, oik = (size_t)s0 * seg_ink, oo = (size_t)s0 * seg_out, ol = (size_t)s0 * seg_lse;
    HA_HOST(cudaMemcpyAsync(dq + oi, static_cast<const char*>(hp->q) + oi, ns * seg_in, cudaMemcpyHostToDevice, ds.copy_in));
    HA_HOST(cudaMemcpyAsync(dk + oik, static_cast<const char*>(hp->k) + oik, ns * seg_ink, cudaMemcpyHostToDevice, ds.copy_in));
    HA_HOST(cudaMemcpyAsync(dv + oik, static_cast<const char*>(hp->v) + oik, ns * seg_ink, cudaMemcpyHostToDevice, ds.copy_in));
    HA_HOST(cudaEventRecord(ds.ev_in[c], ds.copy_in));
    HA_HOST(cudaStreamWaitEvent(st, ds.ev_in[c], 0));
    hyperattn_params p = *hp;
    p.B = 1; p.H = ns;
    p.q = dq + oi; p.k = dk + oik; p.v = dv + oik;
    p.out = dout + oo; p.lse = reinterpret_cast<float*>(dlse + ol);
    rc = forward_impl(p, s0);
    if (rc) return rc;
    HA_HOST(cudaEventRecord(ds.ev_done[c], st));
    HA_HOST(cudaStreamWaitEvent(ds.copy_out, ds.ev_done[c], 0));
    HA_HOST(cudaMemcpyAsync(static_cast<char*>(hp->out) + oo, dout + oo, ns * seg_out, cudaMemcpyDeviceToHost, ds.copy_out));
    HA_HOST(cudaMemcpyAsync(reinterpret_cast<char*>(hp->lse) + ol, dlse + ol, ns * seg_lse, cudaMemcpyDeviceToHost, ds.copy_out));
  }
  // the caller's stream is done when the last results are on the host
  HA_HOST(cudaEventRecord(ds.ev_end, ds.copy_out));
  HA_HOST(cudaStreamWaitEvent(st, ds.ev_end, 0));
#undef HA_HOST
  return HYPERATTN_OK;
}

int hyperattn_workspace_bytes(const hyperattn_params* p, size_t* bytes) {
  if (!p || !bytes) return HYPERATTN_INVALID_ARGUMENT;
  Geometry g;
  const int rc = build_geometry(*p, g);
  if (rc) return rc;
  g.node_dirs = p->node_directions != 0 && g.causal && g.L > 0 && g.sorted;
  *bytes = make_plan(g, p->dtype == HYPERATTN_FP32, 0, p->capped != 0 && g.sorted && g.m > 0,
                     p->sampling == HYPERATTN_SAMPLE_VALUE_NORMS && g.sorted && g.m > 0,
                     p->dtype != HYPERATTN_FP32 && p->out_dtype != HYPERATTN_FP32 && g.L > 0).total;
  return HYPERATTN_OK;
}

int hyperattn_get_projections(int d, int hash_bits, uint64_t seed, float* host_out) {
  if (!host_out || d <= 0 || d > 128 || hash_bits < 1 || hash_bits > 8) return HYPERATTN_INVALID_ARGUMENT;
  make_directions(d, hash_bits, seed, host_out);
  return HYPERATTN_OK;
}

int hyperattn_get_node_projections(int d, int hash_bits, uint64_t seed, int node, float* host_out) {
  if (!host_out || d <= 0 || d > 128 || hash_bits < 1 || hash_bits > 8 || node < 0) return HYPERATTN_INVALID_ARGUMENT;
  make_directions(d, hash_bits, seed, host_out, (uint32_t)node);
  return HYPERATTN_OK;
}

int hyperattn_last_device_status(void* stream, int* status) {
  if (!status) return HYPERATTN_INVALID_ARGUMENT;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceState& ds = g_dev[dev];
  *status = 0;
  if (!ds.status) return HYPERATTN_OK;
  int word = 0;
  if (cudaMemcpy(&word, ds.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (word) {
    if (getenv("HYPERATTN_DEBUG")) std::fprintf(stderr, "hyperattn: device status word %d (site of the wait that gave up)\n", word);
    *status = HYPERATTN_DEVICE_TIMEOUT;
    cudaMemset(ds.status, 0, 4);
  }
  return HYPERATTN_OK;
}

int hyperattn_profile_enable(int on) {
  std::lock_guard<std::mutex> lock(g_mu);
  g_profile = on != 0;
  g_profile_mask = (on == 0 || on == 1) ? ~0u : ((unsigned)on >> 1);
  return HYPERATTN_OK;
}

int hyperattn_profile_reset(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  for (auto& ev : g_events) { g_event_pool.push_back(ev.beg); g_event_pool.push_back(ev.end); }
  g_events.clear();
  g_profile_calls = 0;
  return HYPERATTN_OK;
}

int hyperattn_profile_read(hyperattn_stage_times* out) {
  if (!out) return HYPERATTN_INVALID_ARGUMENT;
  std::lock_guard<std::mutex> lock(g_mu);
  std::memset(out, 0, sizeof(*out));
  for (auto& ev : g_events) {
    if (cudaEventSynchronize(ev.end) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ev.beg, ev.end) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
    out->ms[ev.stage] += ms;
    out->launches[ev.stage] += ev.launches;
  }
  out->calls = g_profile_calls;
  return HYPERATTN_OK;
}

int hyperattn_release(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  int cur = 0;
  cudaGetDevice(&cur);
  for (auto& kv : g_dev) {
    cudaSetDevice(kv.first);
    cudaDeviceSynchronize();
    if (kv.second.ws) cudaFree(kv.second.ws);
    if (kv.second.host_stage) cudaFree(kv.second.host_stage);
    if (kv.second.status) cudaFree(kv.second.status);
    if (kv.second.copy_in) {
      cudaStreamDestroy(kv.second.copy_in); cudaStreamDestroy(kv.second.copy_out);
      cudaEventDestroy(kv.second.ev_start); cudaEventDestroy(kv.second.ev_end);
      for (int c = 0; c < kHostChunks; ++c) { cudaEventDestroy(kv.second.ev_in[c]); cudaEventDestroy(kv.second.ev_done[c]); }
    }
  }
  g_dev.clear();
  for (auto& ev : g_events) { cudaEventDestroy(ev.beg); cudaEventDestroy(ev.end); }
  g_events.clear();
  for (auto& e : g_event_pool) cudaEventDestroy(e);
  g_event_pool.clear();
  cudaSetDevice(cur);
  return HYPERATTN_OK;
}

const char* hyperattn_status_string(int status) {
  switch (status) {
    case HYPERATTN_OK: return "ok";
    case HYPERATTN_INVALID_ARGUMENT: return "invalid argument";
    case HYPERATTN_UNSUPPORTED_SHAPE: return "unsupported shape";
    case HYPERATTN_MISALIGNED: return "misaligned or aliasing pointer";
    case HYPERATTN_WORKSPACE_TOO_SMALL: return "workspace too small";
    case HYPERATTN_CUDA_ERROR: return "CUDA error";
    case HYPERATTN_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int hyperattn_version(void) { return kVersion; }

}  // extern "C"
