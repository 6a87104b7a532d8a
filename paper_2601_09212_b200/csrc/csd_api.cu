// Host side of libcsd: argument checks, workspace layout, launch configuration.
// Every step of the method runs in the kernels of csd_kernels.cuh; nothing here
// touches logits.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/csd.h"
#include "csd_kernels.cuh"
#include "csd_fused.cuh"
#include "csd_tree.cuh"
#include "csd_shard.cuh"

namespace {

using namespace csd;

static_assert(sizeof(TopkSmem) <= 55 * 1024, "four blocks of the top-k kernel per SM must fit");
static_assert(sizeof(TopkSmemT<kWarpListLarge>) <= 56 * 1024, "four blocks of its large-list instance per SM must fit");
static_assert(sizeof(PlainSmem) <= 75 * 1024, "three blocks of the plain kernel per SM must fit");

constexpr int kMaxV = 1 << 20;
constexpr int kMaxDevices = 64;
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int elem_size(int dtype) { return dtype == CSD_F32 ? 4 : 2; }
inline int vec_width(int dtype) { return 16 / elem_size(dtype); }

struct DeviceInfo {
  int sms = 0;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_mutex;

int device_sms(int* dev_out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  if (dev_out) *dev_out = dev;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_dev[dev].sms == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    g_dev[dev].sms = n;
  }
  return g_dev[dev].sms;
}

bool shape_ok(int B, int gamma, int V) {
  return B >= 1 && gamma >= 1 && gamma <= kMaxGamma && V >= 2 && V <= kMaxV;
}

// Workspace: [header: error flag][partials: rows * max_parts float2][thresholds: rows float]
// (the last two: multi-launch path only).  The header must be zero before the first call.
struct Layout {
  size_t rows, max_parts, header_off, partials_off, thresholds_off, zero_bytes, total;
};
Layout layout_for(int B, int gamma, int V, int dtype) {
  Layout l;
  l.rows = (size_t)B * (size_t)(2 * gamma + 1);
  // parts of the multi-launch path (the single-launch path keeps its partials in shared memory)
  const size_t min_part = (size_t)kStatsThreads * vec_width(dtype);  // U = 1
  l.max_parts = ((size_t)V + min_part - 1) / min_part;
  l.header_off = 0;
  l.partials_off = kAlign;
  l.zero_bytes = l.partials_off;
  l.thresholds_off = l.partials_off + align_up(l.rows * l.max_parts * sizeof(float2));
  l.total = l.thresholds_off + align_up(l.rows * sizeof(float));
  return l;
}

// c with P(N(0,1) > c) = tail, by bisection on erfc (host, called once per call; 60 steps)
double normal_upper_quantile(double tail) {
  double lo = -8.0, hi = 8.0;
  for (int it = 0; it < 60; ++it) {
    const double mid = 0.5 * (lo + hi);
    if (0.5 * erfc(mid / sqrt(2.0)) > tail) lo = mid; else hi = mid;
  }
  return 0.5 * (lo + hi);
}

// Launches one of the single-launch kernels (KERNEL: 0 plain, 1 top-k on rows that are a whole
// number of stages, 2 top-k on any row length, 3 and 4 the same two with the large candidate lists) with its shared-memory size, optionally with
// programmatic stream serialisation and as clusters of ctas_per_seq blocks.
template <typename T, bool CFG, int KERNEL>
cudaError_t launch_fused(const FusedArgs& a, int grid, bool overlap, cudaStream_t stream) {
  auto kern = KERNEL == 0 ? verify_plain_kernel<T, CFG>
              : KERNEL == 1 ? verify_topk_kernel<T, CFG, false, kWarpList>
              : KERNEL == 2 ? verify_topk_kernel<T, CFG, true, kWarpList>
              : KERNEL == 3 ? verify_topk_kernel<T, CFG, false, kWarpListLarge>
                            : verify_topk_kernel<T, CFG, true, kWarpListLarge>;
  constexpr size_t kSmem = KERNEL == 0 ? sizeof(PlainSmem) : (KERNEL <= 2 ? sizeof(TopkSmem) : sizeof(TopkSmemT<kWarpListLarge>));
  constexpr int kThreads = KERNEL ? kTopkThreads : kPlainThreads;
  // the attribute belongs to (function, device): set it once per device (setting it twice is harmless)
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n_attr = 0;
  if (overlap) {   // the call may start while the operation before it on the stream is still running
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  if (a.ctas_per_seq > 1) {   // the blocks of a sequence are one cluster
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = (unsigned)a.ctas_per_seq;
    attr[n_attr].val.clusterDim.y = 1;
    attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n_attr;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

template <typename T, bool CFG>
cudaError_t launch_fused_t(const FusedArgs& a, bool topk, int grid, bool overlap, cudaStream_t stream) {
  if (!topk) return launch_fused<T, CFG, 0>(a, grid, overlap, stream);
  constexpr int kStageElems = kTkStageBytes / ((int)sizeof(T) * (CFG ? 2 : 1));
  const bool whole = a.fin.V % kStageElems == 0;
  if (a.large_lists) return whole ? launch_fused<T, CFG, 3>(a, grid, overlap, stream) : launch_fused<T, CFG, 4>(a, grid, overlap, stream);
  return whole ? launch_fused<T, CFG, 1>(a, grid, overlap, stream) : launch_fused<T, CFG, 2>(a, grid, overlap, stream);
}

template <typename T, bool CFG, int U, bool TOPK>
cudaError_t launch_stats(const StatsArgs& a, int sms, cudaStream_t stream) {
  auto kern = row_stats_kernel<T, CFG, U, TOPK>;
  static int cached_per_sm = 0;  // a property of the kernel, the same on every B200
  int per_sm = cached_per_sm;
  if (per_sm == 0) {
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kStatsThreads, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    cached_per_sm = per_sm;
  }
  long long grid = (long long)sms * per_sm;
  if (grid > a.n_items) grid = a.n_items;
  kern<<<(unsigned)grid, kStatsThreads, 0, stream>>>(a);
  return cudaGetLastError();
}

template <typename T, bool CFG>
cudaError_t launch_stats_u(const StatsArgs& a, int U, bool topk, int sms, cudaStream_t stream) {
  if (topk) {  // U is 1 or 4 here
    return U == 4 ? launch_stats<T, CFG, 4, true>(a, sms, stream) : launch_stats<T, CFG, 1, true>(a, sms, stream);
  }
  switch (U) {
    case 8: return launch_stats<T, CFG, 8, false>(a, sms, stream);
    case 4: return launch_stats<T, CFG, 4, false>(a, sms, stream);
    case 2: return launch_stats<T, CFG, 2, false>(a, sms, stream);
    default: return launch_stats<T, CFG, 1, false>(a, sms, stream);
  }
}

template <typename T, bool CFG>
cudaError_t launch_select(const SelectArgs& a, int sms, cudaStream_t stream) {
  const long long rows = (long long)a.B * (a.T + a.gamma);
  long long grid = 2LL * sms;
  if (grid > rows) grid = rows;
  topk_threshold_kernel<T, CFG><<<(unsigned)grid, kSelectThreads, 0, stream>>>(a);
  return cudaGetLastError();
}

template <typename T, bool CFG>
cudaError_t launch_finish(const FinishArgs& a_in, cudaStream_t stream) {
  auto kern = finish_kernel<T, CFG>;
  constexpr int TILE = 32 * Elem<T>::kVec;
  FinishArgs a = a_in;
  size_t slots = (size_t)((a.V + TILE - 1) / TILE);
  if (slots < 2 * (kFinishThreads / 32)) slots = 2 * (kFinishThreads / 32);   // the monitors' two sums per warp
  size_t smem = slots * sizeof(double);
  a.nbr_table_off = 0;
  if (a.nbr != nullptr && smem + (size_t)a.V * sizeof(float) <= 200 * 1024) {   // the similarity relaxation's table of P
    a.nbr_table_off = (int)slots;
    smem += (size_t)a.V * sizeof(float);
  }
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)a.B);
  cfg.blockDim = dim3(kFinishThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

// Test aids (csd_test_hooks): process-wide, read at every launch of the single-launch path.
long long g_wait_limit = kWaitCycles;
int g_drop_first_copy = 0;

// The single-launch path's partition and launch (see the comments inside).  With stats_out set the
// kernels stop after their streaming phase and write every row's (m, s) -- and, with top-k, its exact
// threshold -- to global memory in the row order of the multi-launch kernels (one part per row), for a
// finishing kernel of that path to consume (tree drafts, the similarity relaxation).
struct FusedPlan {
  FinishArgs fa;
  int B, gamma, V, top_k, dtype;
  int rows_per_seq;
  long long rows;
  int sms, es;
  bool cfg, topk, back_to_back, allow_short_cut;
  int* error_flag;
  float2* stats_out;
  float* thr_out;
  cudaStream_t stream;
};
cudaError_t plan_and_launch_fused(const FusedPlan& in) {
  const int sms = in.sms, es = in.es, rows_per_seq = in.rows_per_seq;
  const bool cfg = in.cfg, topk = in.topk;
  cudaStream_t stream = in.stream;
  {
    FusedArgs ua;
    ua.fin = in.fa;
    ua.top_k = in.top_k;
    ua.lo_sigmas = nanf("");
    ua.lo_delta = 0.0f;
    ua.hi_delta = nanf("");
    ua.large_lists = 0;
    ua.error_flag = in.error_flag;
    ua.stats_out = in.stats_out;
    ua.thr_out = in.thr_out;
    ua.wait_limit = g_wait_limit;
    ua.drop_first_copy = g_drop_first_copy;
    // Blocks are aligned with sequences and positions.  For calls enqueued back to back a block owns a
    // whole sequence (for very large batches seqs_per_cta of them): such calls overlap on the GPU as
    // deeply as their grids allow (a call may start once every block of its predecessor has started),
    // so few long-lived blocks per call are best, split only when the batch is too small to give 16
    // blocks.  Otherwise the call runs alone, and a sequence's draft positions are split over the
    // ctas_per_seq blocks of one cluster (each with both rows of its positions; 2, 4 or 8 blocks)
    // until the GPU is full.
    const long long merge_above = 8LL * sms;   // beyond this many sequences a block takes several
    // (measured: the top-k kernel, with its longer per-row work, gains from the finer split)
    const double tk_k = in.top_k, tk_v = in.V;
    const double tk_tail = 1.25 * tk_k / tk_v + 4.0 * sqrt(tk_k) / tk_v + 16.0 / tk_v;
    const bool tk_large = topk && tk_tail * tk_v >= 0.8 * (kTopkWarps * kWarpList);
    const long long split_below = in.back_to_back ? 16 : (topk ? 4LL : 2LL) * sms;
    long long c = 1, spc = 1;
    if (in.B > merge_above) spc = (in.B + merge_above - 1) / merge_above;
    else if (in.B < split_below) {
      const long long want = split_below / in.B;
      while (2 * c <= want && 2 * c <= in.gamma && 2 * c <= kMaxCluster) c *= 2;
    }
    while (spc > 1 && spc * rows_per_seq > kBlockRows) --spc;   // rows_per_seq <= 65 < kBlockRows
    if (topk) {
      ua.chunks_per_part = 0;
      ua.parts_per_row = 1;
      const double k = tk_k, v = tk_v, tail = tk_tail;
      // the candidates must fit the per-warp lists with room to spare: the small lists (four blocks per SM)
      // where they do, else the large ones (three blocks per SM), else every row is selected exactly
      ua.large_lists = tk_large ? 1 : 0;
      if (tail < 0.45 && tail * v < 0.8 * (kTopkWarps * kWarpListLarge)) {
        ua.lo_sigmas = (float)normal_upper_quantile(tail);
        ua.lo_delta = ua.lo_sigmas - (float)normal_upper_quantile(k / v);
        // a level with, almost surely, fewer than k values above it: the mirror image of the guess.
        // The short cut it serves keeps lo as the row's threshold, which the diagnostic outputs that
        // evaluate every token (the distribution drawn from, the monitors) would show in their last
        // digits: with them requested every row gets its exact threshold.
        const double tail_hi = 0.75 * k / v - 4.0 * sqrt(k) / v - 16.0 / v;
        if (tail_hi * v >= 8.0 && in.allow_short_cut)
          ua.hi_delta = (float)normal_upper_quantile(tail_hi) - ua.lo_sigmas;
      }
    } else {
      // warp-wide items: parts of rows, sized so that every warp of the grid gets several
      const int eps = kWStageBytes / (es * (cfg ? 2 : 1));
      const long long cpr = (in.V + eps - 1) / eps;
      // A row is cut into 1 ... 16 parts; the choice minimises the work of the block's busiest warp
      // (its items are a contiguous eighth of the block's items; an item costs its stages plus about
      // half a stage of fixed work).  Long items are better for their own sake -- fewer changes of
      // the running maximum, fewer reductions -- so ties go to the fewer parts.
      const long long rows_b = (c > 1) ? (2LL * ((in.gamma + c - 1) / c) + 1) : spc * rows_per_seq;
      long long cpp = cpr;
      double best = -1.0;
      for (long long np = 1; np <= 16 && np <= cpr; ++np) {
        const long long cand = (cpr + np - 1) / np;          // stages per part
        const long long parts = (cpr + cand - 1) / cand;
        if (parts != np && np > 1) continue;                 // (the same cut as a smaller np)
        const long long n = rows_b * parts;
        const long long last = cpr - (parts - 1) * cand;      // stages of a row's last part
        double worst = 0.0;
        for (int w = 0; w < kPlainWarps; ++w) {
          const long long b0 = n * w / kPlainWarps, b1 = n * (w + 1) / kPlainWarps;
          // items b0 .. b1-1; item i is part i % parts of its row
          const long long full_rows = (b1 - b0) / parts;
          double load = (double)full_rows * ((double)cpr + 0.5 * (double)parts);
          for (long long i = b0 + full_rows * parts; i < b1; ++i)
            load += (double)((i % parts == parts - 1) ? last : cand) + 0.5;
          if (load > worst) worst = load;
        }
        if (best < 0.0 || worst < best * 0.97) { best = worst; cpp = cand; }
      }
      // a block keeps one stash entry per item
      for (;;) {
        const long long parts = (cpr + cpp - 1) / cpp;
        const long long rows_block = (c > 1) ? (2LL * ((in.gamma + c - 1) / c) + 1) : spc * rows_per_seq;
        if (rows_block * parts <= kBlockStash) break;
        if (cpp < cpr) cpp = (cpp * 2 < cpr) ? cpp * 2 : cpr;
        else if (spc > 1) --spc;
        else break;   // one sequence per block, one part per row: at most 65 items
      }
      ua.chunks_per_part = (int)cpp;
      ua.parts_per_row = (int)((cpr + cpp - 1) / cpp);
    }
    const long long grid = c > 1 ? (long long)in.B * c : (in.B + spc - 1) / spc;
    ua.ctas_per_seq = (int)c;
    ua.seqs_per_cta = (int)spc;
    cudaError_t fe;
    const bool overlap = in.back_to_back != 0;
    if (in.dtype == CSD_F32)
      fe = cfg ? launch_fused_t<float, true>(ua, topk, (int)grid, overlap, stream)
               : launch_fused_t<float, false>(ua, topk, (int)grid, overlap, stream);
    else
      fe = cfg ? launch_fused_t<__nv_bfloat16, true>(ua, topk, (int)grid, overlap, stream)
               : launch_fused_t<__nv_bfloat16, false>(ua, topk, (int)grid, overlap, stream);
    return fe;
  }
}

// sampling: the degenerate round used by csd_sample_rows -- no draft positions (gamma = 0), one
// "target" row per sequence, whose bonus draw is the wanted token; the drafter-side pointers are unused.
// no_workspace: the call has no workspace (the simple forms): only the single-launch path, which keeps
// nothing in global memory, can serve it; otherwise CSD_ERR_ALIGN.
// similar: the similarity relaxation's neighbour table (csd_verify_similar); served by the multi-launch path.
struct Similar {
  const int32_t* nbr = nullptr;
  int k = 0;
  float lambda = 0.0f;
};
int verify_impl(const csd_params& p, int* plan_only = nullptr, bool sampling = false, bool no_workspace = false,
                const Similar& similar = Similar()) {
  if (sampling) {
    if (!p.target_logits || !p.uniforms || !p.out_tokens) return CSD_ERR_NULL;
  } else if (!p.target_logits || !p.draft_logits || !p.draft_tokens || !p.uniforms || !p.relax_schedule ||
             !p.out_tokens || !p.out_accept_len) {
    return CSD_ERR_NULL;
  }
  if (p.dtype != CSD_F32 && p.dtype != CSD_BF16) return CSD_ERR_DTYPE;
  if (sampling) {
    if (p.B < 1 || p.gamma != 0 || p.target_rows != 1 || p.V < 2 || p.V > kMaxV) return CSD_ERR_SHAPE;
  } else if (!shape_ok(p.B, p.gamma, p.V)) {
    return CSD_ERR_SHAPE;
  }
  if (p.target_rows != p.gamma && p.target_rows != p.gamma + 1) return CSD_ERR_SHAPE;
  const int64_t tstride = p.target_batch_stride ? p.target_batch_stride : (int64_t)p.target_rows * p.V;
  const int64_t dstride = p.draft_batch_stride ? p.draft_batch_stride : (int64_t)p.gamma * p.V;
  if (tstride < (int64_t)p.target_rows * p.V || dstride < (int64_t)p.gamma * p.V) return CSD_ERR_SHAPE;
  const bool cfg = p.target_uncond != nullptr;
  if ((p.target_uncond == nullptr) != (p.draft_uncond == nullptr)) return CSD_ERR_ARG;
  if (p.top_k < 0) return CSD_ERR_ARG;
  if (cfg && !isfinite(p.cfg_scale)) return CSD_ERR_ARG;
  const bool topk = p.top_k > 0 && p.top_k < p.V;
  const Layout lay = layout_for(p.B, p.gamma, p.V, p.dtype);
  if (!no_workspace && (!p.workspace || ((uintptr_t)p.workspace % kAlign) != 0 || p.workspace_bytes < lay.total))
    return CSD_ERR_WORKSPACE;
  int dev = 0;
  const int sms = device_sms(&dev);
  if (sms <= 0) return CSD_ERR_LAUNCH;

  const int es = elem_size(p.dtype), vw = vec_width(p.dtype);
  auto aligned16 = [](const void* q) { return ((uintptr_t)q & 15u) == 0; };
  bool vec_ok = (p.V % vw) == 0 && (tstride * es) % 16 == 0 && (dstride * es) % 16 == 0 &&
                aligned16(p.target_logits) && aligned16(p.draft_logits);
  if (cfg) vec_ok = vec_ok && aligned16(p.target_uncond) && aligned16(p.draft_uncond);

  cudaStream_t stream = (cudaStream_t)p.stream;
  const int rows_per_seq = p.target_rows + p.gamma;
  const long long rows = (long long)p.B * rows_per_seq;

  // part size: the largest that still leaves every SM several blocks to work on
  int U = (cfg || topk) ? 4 : 8;
  auto parts_for = [&](int u) { return (p.V + kStatsThreads * u * vw - 1) / (kStatsThreads * u * vw); };
  while (U > 1 && rows * parts_for(U) < 4LL * sms) U >>= 1;
  if (topk && U == 2) U = 1;

  StatsArgs sa;
  sa.target = p.target_logits; sa.draft = p.draft_logits;
  sa.target_uncond = p.target_uncond; sa.draft_uncond = p.draft_uncond;
  sa.cfg_scale = p.cfg_scale;
  sa.B = p.B; sa.gamma = p.gamma; sa.T = p.target_rows; sa.V = p.V;
  sa.tstride = tstride; sa.dstride = dstride;
  sa.parts = parts_for(U);
  sa.part_elems = kStatsThreads * U * vw;
  sa.n_items = (int)(rows * sa.parts);
  sa.vec_ok = vec_ok ? 1 : 0;
  char* const ws = no_workspace ? nullptr : (char*)p.workspace;   // (the single-launch path never touches these)
  sa.partials = ws ? reinterpret_cast<float2*>(ws + lay.partials_off) : nullptr;
  sa.thresholds = ws ? reinterpret_cast<const float*>(ws + lay.thresholds_off) : nullptr;

  SelectArgs se;
  se.target = p.target_logits; se.draft = p.draft_logits;
  se.target_uncond = p.target_uncond; se.draft_uncond = p.draft_uncond;
  se.cfg_scale = p.cfg_scale;
  se.B = p.B; se.gamma = p.gamma; se.T = p.target_rows; se.V = p.V;
  se.tstride = tstride; se.dstride = dstride;
  se.vec_ok = sa.vec_ok;
  se.top_k = p.top_k;
  se.thresholds = ws ? reinterpret_cast<float*>(ws + lay.thresholds_off) : nullptr;

  FinishArgs fa;
  fa.target = p.target_logits; fa.draft = p.draft_logits;
  fa.target_uncond = p.target_uncond; fa.draft_uncond = p.draft_uncond;
  fa.cfg_scale = p.cfg_scale;
  fa.B = p.B; fa.gamma = p.gamma; fa.T = p.target_rows; fa.V = p.V;
  fa.tstride = tstride; fa.dstride = dstride;
  fa.parts = sa.parts;
  fa.vec_ok = sa.vec_ok;
  fa.use_topk = topk ? 1 : 0;
  fa.partials = sa.partials;
  fa.thresholds = sa.thresholds;
  fa.tokens = p.draft_tokens; fa.uniforms = p.uniforms; fa.schedule = p.relax_schedule;
  fa.out_tokens = p.out_tokens; fa.out_accept_len = p.out_accept_len; fa.out_status = p.out_status;
  fa.dbg_p = p.dbg_p; fa.dbg_q = p.dbg_q; fa.dbg_f = p.dbg_f; fa.dbg_G = p.dbg_G;
  fa.diag_am = p.diag_accept_mass; fa.diag_bt = p.diag_bound_term;
  fa.nbr = similar.nbr; fa.nbr_k = similar.k; fa.nbr_lambda = similar.lambda;

  // ---- fused single-launch path: aligned rows of at least 512 bytes; with top-k, rows that fit the registers
  const bool fused = vec_ok && (size_t)p.V * es >= 512 && (p.V + 32 * vw - 1) / (32 * vw) <= kFinTiles &&
                     similar.nbr == nullptr;
  if (no_workspace && !fused) return CSD_ERR_ALIGN;
  // the similarity relaxation finishes in the multi-launch path's kernel; where the rows qualify, their
  // statistics still come from the streaming kernels (one launch, every logit read once)
  const bool stream_stats = !fused && similar.nbr != nullptr && !no_workspace && vec_ok && (size_t)p.V * es >= 512 &&
                            (p.V + 32 * vw - 1) / (32 * vw) <= kFinTiles;
  if (plan_only) {  // number of kernels this call would enqueue
    *plan_only = fused ? 1 : (stream_stats ? 2 : (topk ? 3 : 2));
    return CSD_OK;
  }
  if (fused) {
    FusedPlan fp;
    fp.fa = fa;
    fp.B = p.B; fp.gamma = p.gamma; fp.V = p.V; fp.top_k = p.top_k; fp.dtype = p.dtype;
    fp.rows_per_seq = rows_per_seq; fp.rows = rows; fp.sms = sms; fp.es = es;
    fp.cfg = cfg; fp.topk = topk; fp.back_to_back = p.back_to_back != 0;
    fp.allow_short_cut = !p.dbg_G && !p.diag_accept_mass && !p.diag_bound_term;
    fp.error_flag = no_workspace ? nullptr : reinterpret_cast<int*>((char*)p.workspace + lay.header_off);
    fp.stats_out = nullptr; fp.thr_out = nullptr;
    fp.stream = stream;
    return plan_and_launch_fused(fp) == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
  }

  cudaError_t e = cudaSuccess;
  if (stream_stats) {
    FusedPlan fp;
    fa.parts = 1;
    fp.fa = fa;
    fp.B = p.B; fp.gamma = p.gamma; fp.V = p.V; fp.top_k = p.top_k; fp.dtype = p.dtype;
    fp.rows_per_seq = rows_per_seq; fp.rows = rows; fp.sms = sms; fp.es = es;
    fp.cfg = cfg; fp.topk = topk; fp.back_to_back = false;
    fp.allow_short_cut = false;   // the finishing kernel filters by the exact threshold
    fp.error_flag = reinterpret_cast<int*>((char*)p.workspace + lay.header_off);
    fp.stats_out = sa.partials;
    fp.thr_out = topk ? se.thresholds : nullptr;
    fp.stream = stream;
    e = plan_and_launch_fused(fp);
    if (e == cudaSuccess) {
      if (p.dtype == CSD_F32) e = cfg ? launch_finish<float, true>(fa, stream) : launch_finish<float, false>(fa, stream);
      else e = cfg ? launch_finish<__nv_bfloat16, true>(fa, stream) : launch_finish<__nv_bfloat16, false>(fa, stream);
    }
  } else if (p.dtype == CSD_F32) {
    if (topk) e = cfg ? launch_select<float, true>(se, sms, stream) : launch_select<float, false>(se, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_stats_u<float, true>(sa, U, topk, sms, stream) : launch_stats_u<float, false>(sa, U, topk, sms, stream);
    if (e == cudaSuccess) e = cfg ? launch_finish<float, true>(fa, stream) : launch_finish<float, false>(fa, stream);
  } else {
    if (topk)
      e = cfg ? launch_select<__nv_bfloat16, true>(se, sms, stream) : launch_select<__nv_bfloat16, false>(se, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_stats_u<__nv_bfloat16, true>(sa, U, topk, sms, stream)
              : launch_stats_u<__nv_bfloat16, false>(sa, U, topk, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_finish<__nv_bfloat16, true>(fa, stream) : launch_finish<__nv_bfloat16, false>(fa, stream);
  }
  return e == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

}  // namespace

extern "C" {

size_t csd_workspace_size(int B, int gamma, int V, int dtype) {
  if (!shape_ok(B, gamma, V) || (dtype != CSD_F32 && dtype != CSD_BF16)) return 0;
  return layout_for(B, gamma, V, dtype).total;
}

int csd_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return CSD_ERR_NULL;
  if (((uintptr_t)workspace % kAlign) != 0 || workspace_bytes == 0) return CSD_ERR_WORKSPACE;
  return cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream) == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

int csd_launch_count(const csd_params* p) {
  if (!p) return CSD_ERR_NULL;
  int n = 0;
  const int rc = verify_impl(*p, &n);
  return rc == CSD_OK ? n : rc;
}

int csd_verify_ex(const csd_params* p) {
  if (!p) return CSD_ERR_NULL;
  return verify_impl(*p);
}

size_t csd_sample_workspace_size(int R, int V, int dtype) {
  if (R < 1 || V < 2 || V > kMaxV || (dtype != CSD_F32 && dtype != CSD_BF16)) return 0;
  return layout_for(R, 0, V, dtype).total;
}

int csd_sample_rows(const void* logits, const void* uncond, float cfg_scale, int top_k, int dtype, int R, int V,
                    int64_t row_stride, const float* uniforms, int32_t* out_tokens, int32_t* out_status,
                    void* workspace, size_t workspace_bytes, int back_to_back, void* stream) {
  csd_params p;
  memset(&p, 0, sizeof p);
  p.target_logits = logits;
  p.draft_logits = logits;       // unused: there are no draft positions
  p.target_uncond = uncond;
  p.draft_uncond = uncond;
  p.cfg_scale = cfg_scale;
  p.top_k = top_k;
  p.dtype = dtype;
  p.B = R; p.gamma = 0; p.V = V; p.target_rows = 1;
  p.target_batch_stride = row_stride;
  p.uniforms = uniforms;         // [R]: the round's layout [B, gamma + 1] with gamma = 0
  p.out_tokens = out_tokens;     // [R]: the round's layout [B, gamma + 1]
  p.out_status = out_status;
  p.workspace = workspace;
  p.workspace_bytes = workspace_bytes;
  p.back_to_back = back_to_back;
  p.stream = stream;
  return verify_impl(p, nullptr, true);
}

int csd_verify(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
               const float* uniforms, const float* relax_schedule, int B, int gamma, int V,
               int32_t* out_tokens, int32_t* out_accept_len, void* stream) {
  if (!shape_ok(B, gamma, V)) return CSD_ERR_SHAPE;
  csd_params p;
  memset(&p, 0, sizeof p);
  p.target_logits = target_logits; p.draft_logits = draft_logits;
  p.cfg_scale = 1.0f; p.top_k = 0; p.dtype = CSD_F32;
  p.B = B; p.gamma = gamma; p.V = V; p.target_rows = gamma;
  p.draft_tokens = draft_tokens; p.uniforms = uniforms; p.relax_schedule = relax_schedule;
  p.out_tokens = out_tokens; p.out_accept_len = out_accept_len;
  p.stream = stream;
  return verify_impl(p, nullptr, false, /*no_workspace=*/true);
}

int csd_verify_similar(const csd_params* p, const int32_t* neighbours, int k, float lambda) {
  if (!p || !neighbours) return CSD_ERR_NULL;
  if (k < 1 || k > 64 || !(lambda >= 0.0f) || !isfinite(lambda)) return CSD_ERR_ARG;
  if (p->diag_accept_mass || p->diag_bound_term) return CSD_ERR_ARG;   // (the monitors are those of Eq. relax)
  Similar sim;
  sim.nbr = neighbours; sim.k = k; sim.lambda = lambda;
  return verify_impl(*p, nullptr, false, false, sim);
}

int csd_checked_report(int32_t* out_host) {
  if (!out_host) return CSD_ERR_NULL;
  int32_t v[4] = {0, 0, 0, 0};
  if (cudaMemcpyFromSymbol(v, g_checked, sizeof v) != cudaSuccess) return CSD_ERR_LAUNCH;
  for (int k = 0; k < 4; ++k) out_host[k] = v[k];
#ifdef CSD_CHECKED
  return 1;
#else
  return 0;
#endif
}

int csd_test_hooks(int wait_limit_log2_cycles, int drop_first_copy) {
  if (wait_limit_log2_cycles != 0 && (wait_limit_log2_cycles < 10 || wait_limit_log2_cycles > 40)) return CSD_ERR_ARG;
  g_wait_limit = wait_limit_log2_cycles ? (1ll << wait_limit_log2_cycles) : kWaitCycles;
  g_drop_first_copy = drop_first_copy ? 1 : 0;
  return CSD_OK;
}

// ---- tree-structured verification ---------------------------------------------------------
}  // extern "C"
namespace {
template <typename T, bool CFG>
cudaError_t launch_tree_finish(const TreeArgs& a_in, cudaStream_t stream) {
  auto kern = tree_finish_kernel<T, CFG>;
  constexpr int TILE = 32 * Elem<T>::kVec;
  TreeArgs a = a_in;
  size_t slots = (size_t)((a.fin.V + TILE - 1) / TILE);
  if (slots < 64) slots = 64;
  size_t smem = slots * sizeof(double);
  a.tab_off = 0;
  if (smem + 2 * (size_t)a.fin.V * sizeof(float) <= 200 * 1024) {   // the walk's tables of the residual and of Q
    a.tab_off = (int)slots;
    smem += 2 * (size_t)a.fin.V * sizeof(float);
  }
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)a.fin.B);
  cfg.blockDim = dim3(kFinishThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

// Depth of the tree (the root's children are level 1), or a negative csd_error for a malformed one:
// a parent that is not -1 or an earlier node, more than kMaxSiblings children of one node, a level
// beyond kMaxTreeDepth.
int tree_depth_checked(const int32_t* parent, int N) {
  if (!parent) return CSD_ERR_NULL;
  if (N < 1 || N > kMaxTreeNodes) return CSD_ERR_SHAPE;
  int level[kMaxTreeNodes], kids[kMaxTreeNodes + 1];
  memset(kids, 0, sizeof kids);
  int D = 0;
  for (int n = 0; n < N; ++n) {
    if (parent[n] < -1 || parent[n] >= n) return CSD_ERR_ARG;
    level[n] = parent[n] < 0 ? 1 : level[parent[n]] + 1;
    if (level[n] > kMaxTreeDepth) return CSD_ERR_SHAPE;
    if (++kids[parent[n] + 1] > kMaxSiblings) return CSD_ERR_SHAPE;
    if (level[n] > D) D = level[n];
  }
  return D;
}
}  // namespace
extern "C" {

int csd_tree_depth(const int32_t* parent_host, int N) { return tree_depth_checked(parent_host, N); }

size_t csd_tree_workspace_size(int B, int N, int V, int dtype) {
  if (B < 1 || N < 1 || N > kMaxTreeNodes || V < 2 || V > kMaxV || (dtype != CSD_F32 && dtype != CSD_BF16)) return 0;
  return layout_for(B, N + 1, V, dtype).total;
}

int csd_verify_tree(const csd_tree_params* pp) {
  if (!pp) return CSD_ERR_NULL;
  const csd_tree_params& p = *pp;
  if (!p.target_logits || !p.draft_logits || !p.parent || !p.draft_tokens || !p.uniforms || !p.relax_schedule ||
      !p.out_tokens || !p.out_accept_len)
    return CSD_ERR_NULL;
  if (p.dtype != CSD_F32 && p.dtype != CSD_BF16) return CSD_ERR_DTYPE;
  if (p.B < 1 || p.V < 2 || p.V > kMaxV) return CSD_ERR_SHAPE;
  const int D = tree_depth_checked(p.parent, p.N);
  if (D < 0) return D;
  if ((p.target_uncond == nullptr) != (p.draft_uncond == nullptr)) return CSD_ERR_ARG;
  if (p.top_k < 0) return CSD_ERR_ARG;
  const bool cfg = p.target_uncond != nullptr;
  if (cfg && !isfinite(p.cfg_scale)) return CSD_ERR_ARG;
  const bool topk = p.top_k > 0 && p.top_k < p.V;
  const int C = p.N + 1;
  const Layout lay = layout_for(p.B, C, p.V, p.dtype);
  if (!p.workspace || ((uintptr_t)p.workspace % kAlign) != 0 || p.workspace_bytes < lay.total) return CSD_ERR_WORKSPACE;
  const int sms = device_sms(nullptr);
  if (sms <= 0) return CSD_ERR_LAUNCH;
  const int es = elem_size(p.dtype), vw = vec_width(p.dtype);
  auto aligned16 = [](const void* q) { return ((uintptr_t)q & 15u) == 0; };
  const int64_t stride = (int64_t)C * p.V;
  bool vec_ok = (p.V % vw) == 0 && (stride * es) % 16 == 0 && aligned16(p.target_logits) && aligned16(p.draft_logits);
  if (cfg) vec_ok = vec_ok && aligned16(p.target_uncond) && aligned16(p.draft_uncond);
  cudaStream_t stream = (cudaStream_t)p.stream;
  const long long rows = (long long)p.B * 2 * C;
  int U = (cfg || topk) ? 4 : 8;
  auto parts_for = [&](int u) { return (p.V + kStatsThreads * u * vw - 1) / (kStatsThreads * u * vw); };
  while (U > 1 && rows * parts_for(U) < 4LL * sms) U >>= 1;
  if (topk && U == 2) U = 1;
  char* const ws = (char*)p.workspace;

  // the row statistics see a chain of C positions with C target rows
  StatsArgs sa;
  sa.target = p.target_logits; sa.draft = p.draft_logits;
  sa.target_uncond = p.target_uncond; sa.draft_uncond = p.draft_uncond;
  sa.cfg_scale = p.cfg_scale;
  sa.B = p.B; sa.gamma = C; sa.T = C; sa.V = p.V;
  sa.tstride = stride; sa.dstride = stride;
  sa.parts = parts_for(U);
  sa.part_elems = kStatsThreads * U * vw;
  sa.n_items = (int)(rows * sa.parts);
  sa.vec_ok = vec_ok ? 1 : 0;
  sa.partials = reinterpret_cast<float2*>(ws + lay.partials_off);
  sa.thresholds = reinterpret_cast<const float*>(ws + lay.thresholds_off);
  SelectArgs se;
  se.target = p.target_logits; se.draft = p.draft_logits;
  se.target_uncond = p.target_uncond; se.draft_uncond = p.draft_uncond;
  se.cfg_scale = p.cfg_scale;
  se.B = p.B; se.gamma = C; se.T = C; se.V = p.V;
  se.tstride = stride; se.dstride = stride;
  se.vec_ok = sa.vec_ok;
  se.top_k = p.top_k;
  se.thresholds = reinterpret_cast<float*>(ws + lay.thresholds_off);
  TreeArgs ta;
  memset(&ta, 0, sizeof ta);
  FinishArgs& fa = ta.fin;
  fa.target = p.target_logits; fa.draft = p.draft_logits;
  fa.target_uncond = p.target_uncond; fa.draft_uncond = p.draft_uncond;
  fa.cfg_scale = p.cfg_scale;
  fa.B = p.B; fa.gamma = C; fa.T = C; fa.V = p.V;
  fa.tstride = stride; fa.dstride = stride;
  fa.parts = sa.parts;
  fa.vec_ok = sa.vec_ok;
  fa.use_topk = topk ? 1 : 0;
  fa.partials = sa.partials;
  fa.thresholds = sa.thresholds;
  fa.tokens = p.draft_tokens; fa.uniforms = p.uniforms; fa.schedule = p.relax_schedule;
  fa.out_tokens = p.out_tokens; fa.out_accept_len = p.out_accept_len; fa.out_status = p.out_status;
  fa.dbg_G = p.dbg_G;
  ta.N = p.N; ta.D = D;
  ta.out_nodes = p.out_nodes;
  for (int n = 0; n < p.N; ++n) ta.parent[n] = (signed char)p.parent[n];

  cudaError_t e = cudaSuccess;
  // Row statistics (and thresholds) of all 2 C rows: by the streaming kernels of the single-launch path
  // where the rows qualify for them (aligned, at least 512 bytes, within the draw's tile table), one
  // launch that reads every logit once; otherwise by the select and statistics kernels.
  const bool stream_stats = vec_ok && (size_t)p.V * es >= 512 && (p.V + 32 * vw - 1) / (32 * vw) <= kFinTiles &&
                            2 * C <= kBlockRows;
  if (stream_stats) {
    FusedPlan fp;
    fp.fa = fa;
    fp.fa.parts = 1;
    fp.B = p.B; fp.gamma = C; fp.V = p.V; fp.top_k = p.top_k; fp.dtype = p.dtype;
    fp.rows_per_seq = 2 * C; fp.rows = rows; fp.sms = sms; fp.es = es;
    fp.cfg = cfg; fp.topk = topk; fp.back_to_back = false;
    fp.allow_short_cut = false;   // the finishing kernel filters by the exact threshold
    fp.error_flag = reinterpret_cast<int*>(ws + lay.header_off);
    fp.stats_out = sa.partials;
    fp.thr_out = topk ? se.thresholds : nullptr;
    fp.stream = stream;
    e = plan_and_launch_fused(fp);
    fa.parts = 1;
    if (e == cudaSuccess) {
      if (p.dtype == CSD_F32) e = cfg ? launch_tree_finish<float, true>(ta, stream) : launch_tree_finish<float, false>(ta, stream);
      else e = cfg ? launch_tree_finish<__nv_bfloat16, true>(ta, stream) : launch_tree_finish<__nv_bfloat16, false>(ta, stream);
    }
  } else if (p.dtype == CSD_F32) {
    if (topk) e = cfg ? launch_select<float, true>(se, sms, stream) : launch_select<float, false>(se, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_stats_u<float, true>(sa, U, topk, sms, stream) : launch_stats_u<float, false>(sa, U, topk, sms, stream);
    if (e == cudaSuccess) e = cfg ? launch_tree_finish<float, true>(ta, stream) : launch_tree_finish<float, false>(ta, stream);
  } else {
    if (topk)
      e = cfg ? launch_select<__nv_bfloat16, true>(se, sms, stream) : launch_select<__nv_bfloat16, false>(se, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_stats_u<__nv_bfloat16, true>(sa, U, topk, sms, stream)
              : launch_stats_u<__nv_bfloat16, false>(sa, U, topk, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_tree_finish<__nv_bfloat16, true>(ta, stream) : launch_tree_finish<__nv_bfloat16, false>(ta, stream);
  }
  return e == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

// ---- vocabulary-sharded verification --------------------------------------------------------
}  // extern "C"
namespace {
struct ShardLayout {
  size_t parts, partials_off, tiles_off, ctx_off, total;
  int U;
};
ShardLayout shard_layout(int B, int gamma, int T, int Vs, int dtype, bool cfg, int sms) {
  ShardLayout l;
  const int vw = vec_width(dtype);
  const long long rows = (long long)B * (T + gamma);
  int U = cfg ? 4 : 8;
  auto parts_for = [&](int u) { return (Vs + kStatsThreads * u * vw - 1) / (kStatsThreads * u * vw); };
  while (U > 1 && sms > 0 && rows * parts_for(U) < 4LL * sms) U >>= 1;
  l.U = U;
  l.parts = (size_t)parts_for(1);   // sized for the finest split, whatever the device
  const size_t ntiles = ((size_t)Vs + 32 * vw - 1) / (32 * vw);
  l.partials_off = 0;
  l.tiles_off = align_up((size_t)rows * l.parts * sizeof(float2));
  l.ctx_off = l.tiles_off + align_up((size_t)B * ntiles * sizeof(double));
  l.total = l.ctx_off + align_up((size_t)B * 64);
  return l;
}

int shard_check(const csd_shard_params& p) {
  if (!p.target_logits || !p.draft_logits || !p.draft_tokens || !p.uniforms || !p.relax_schedule) return CSD_ERR_NULL;
  if (p.dtype != CSD_F32 && p.dtype != CSD_BF16) return CSD_ERR_DTYPE;
  if (p.B < 1 || p.gamma < 1 || p.gamma > kMaxGamma || p.Vs < 1 || p.Vs > kMaxV) return CSD_ERR_SHAPE;
  if (p.target_rows != p.gamma && p.target_rows != p.gamma + 1) return CSD_ERR_SHAPE;
  if (p.n_shards < 1 || p.n_shards > 1024 || p.shard < 0 || p.shard >= p.n_shards) return CSD_ERR_SHAPE;
  if (p.v_offset < 0 || p.V_total < 2 || (long long)p.v_offset + p.Vs > p.V_total) return CSD_ERR_SHAPE;
  if ((p.target_uncond == nullptr) != (p.draft_uncond == nullptr)) return CSD_ERR_ARG;
  if (p.target_uncond && !isfinite(p.cfg_scale)) return CSD_ERR_ARG;
  const ShardLayout lay = shard_layout(p.B, p.gamma, p.target_rows, p.Vs, p.dtype, p.target_uncond != nullptr, 0);
  if (!p.workspace || ((uintptr_t)p.workspace % kAlign) != 0 || p.workspace_bytes < lay.total) return CSD_ERR_WORKSPACE;
  return CSD_OK;
}

// the slice as the kernels see it
void shard_args(const csd_shard_params& p, int sms, ShardArgs& sa, StatsArgs& st) {
  const bool cfg = p.target_uncond != nullptr;
  const ShardLayout lay = shard_layout(p.B, p.gamma, p.target_rows, p.Vs, p.dtype, cfg, sms);
  const int es = elem_size(p.dtype), vw = vec_width(p.dtype);
  auto aligned16 = [](const void* q) { return ((uintptr_t)q & 15u) == 0; };
  const int64_t tstride = (int64_t)p.target_rows * p.Vs, dstride = (int64_t)p.gamma * p.Vs;
  bool vec_ok = (p.Vs % vw) == 0 && (tstride * es) % 16 == 0 && (dstride * es) % 16 == 0 &&
                aligned16(p.target_logits) && aligned16(p.draft_logits);
  if (cfg) vec_ok = vec_ok && aligned16(p.target_uncond) && aligned16(p.draft_uncond);
  char* ws = (char*)p.workspace;
  memset(&sa, 0, sizeof sa);
  FinishArgs& f = sa.fin;
  f.target = p.target_logits; f.draft = p.draft_logits;
  f.target_uncond = p.target_uncond; f.draft_uncond = p.draft_uncond;
  f.cfg_scale = p.cfg_scale;
  f.B = p.B; f.gamma = p.gamma; f.T = p.target_rows; f.V = p.Vs;
  f.tstride = tstride; f.dstride = dstride;
  f.parts = (p.Vs + kStatsThreads * lay.U * vw - 1) / (kStatsThreads * lay.U * vw);
  f.vec_ok = vec_ok ? 1 : 0;
  f.partials = reinterpret_cast<const float2*>(ws + lay.partials_off);
  f.tokens = p.draft_tokens; f.uniforms = p.uniforms; f.schedule = p.relax_schedule;
  sa.n_shards = p.n_shards; sa.shard = p.shard; sa.v_offset = p.v_offset; sa.V_total = p.V_total;
  sa.tile_sums = reinterpret_cast<double*>(ws + lay.tiles_off);
  sa.ctx = reinterpret_cast<float4*>(ws + lay.ctx_off);
  st.target = p.target_logits; st.draft = p.draft_logits;
  st.target_uncond = p.target_uncond; st.draft_uncond = p.draft_uncond;
  st.cfg_scale = p.cfg_scale;
  st.B = p.B; st.gamma = p.gamma; st.T = p.target_rows; st.V = p.Vs;
  st.tstride = tstride; st.dstride = dstride;
  st.parts = f.parts;
  st.part_elems = kStatsThreads * lay.U * vw;
  st.n_items = (int)((long long)p.B * (p.target_rows + p.gamma) * st.parts);
  st.vec_ok = f.vec_ok;
  st.partials = reinterpret_cast<float2*>(ws + lay.partials_off);
  st.thresholds = nullptr;
}

template <typename K>
cudaError_t launch_after(K kern, const ShardArgs& a, unsigned grid, unsigned block, cudaStream_t stream) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}
}  // namespace
extern "C" {

size_t csd_shard_workspace_size(int B, int gamma, int target_rows, int Vs, int dtype) {
  if (B < 1 || gamma < 1 || gamma > kMaxGamma || Vs < 1 || Vs > kMaxV || (dtype != CSD_F32 && dtype != CSD_BF16)) return 0;
  if (target_rows != gamma && target_rows != gamma + 1) return 0;
  return shard_layout(B, gamma, target_rows, Vs, dtype, false, 0).total;
}

int csd_shard_stats(const csd_shard_params* pp, void* out_records) {
  if (!pp || !out_records) return CSD_ERR_NULL;
  const csd_shard_params& p = *pp;
  const int rc = shard_check(p);
  if (rc != CSD_OK) return rc;
  const int sms = device_sms(nullptr);
  if (sms <= 0) return CSD_ERR_LAUNCH;
  ShardArgs sa; StatsArgs st;
  shard_args(p, sms, sa, st);
  sa.local = reinterpret_cast<float4*>(out_records);
  const bool cfg = p.target_uncond != nullptr;
  const int U = st.part_elems / (kStatsThreads * vec_width(p.dtype));
  cudaStream_t stream = (cudaStream_t)p.stream;
  const unsigned grid = (unsigned)((p.B * (p.target_rows + p.gamma) + 7) / 8);
  cudaError_t e;
  if (p.dtype == CSD_F32) {
    e = cfg ? launch_stats_u<float, true>(st, U, false, sms, stream) : launch_stats_u<float, false>(st, U, false, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_after(shard_merge_kernel<float, true>, sa, grid, 256, stream)
              : launch_after(shard_merge_kernel<float, false>, sa, grid, 256, stream);
  } else {
    e = cfg ? launch_stats_u<__nv_bfloat16, true>(st, U, false, sms, stream)
            : launch_stats_u<__nv_bfloat16, false>(st, U, false, sms, stream);
    if (e == cudaSuccess)
      e = cfg ? launch_after(shard_merge_kernel<__nv_bfloat16, true>, sa, grid, 256, stream)
              : launch_after(shard_merge_kernel<__nv_bfloat16, false>, sa, grid, 256, stream);
  }
  return e == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

int csd_shard_partial(const csd_shard_params* pp, const void* records_all, double* out_totals, float* dbg_p, float* dbg_q,
                      float* dbg_f) {
  if (!pp || !records_all || !out_totals) return CSD_ERR_NULL;
  const csd_shard_params& p = *pp;
  const int rc = shard_check(p);
  if (rc != CSD_OK) return rc;
  ShardArgs sa; StatsArgs st;
  shard_args(p, device_sms(nullptr), sa, st);
  sa.gathered = reinterpret_cast<const float4*>(records_all);
  sa.z_local = out_totals;
  sa.fin.dbg_p = dbg_p; sa.fin.dbg_q = dbg_q; sa.fin.dbg_f = dbg_f;
  const bool cfg = p.target_uncond != nullptr;
  cudaStream_t stream = (cudaStream_t)p.stream;
  if (p.dtype == CSD_F32) {
    if (cfg) shard_partial_kernel<float, true><<<p.B, kFinishThreads, 0, stream>>>(sa);
    else shard_partial_kernel<float, false><<<p.B, kFinishThreads, 0, stream>>>(sa);
  } else {
    if (cfg) shard_partial_kernel<__nv_bfloat16, true><<<p.B, kFinishThreads, 0, stream>>>(sa);
    else shard_partial_kernel<__nv_bfloat16, false><<<p.B, kFinishThreads, 0, stream>>>(sa);
  }
  return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

int csd_shard_pick(const csd_shard_params* pp, const void* records_all, const double* totals_all, int32_t* out_candidates) {
  if (!pp || !records_all || !totals_all || !out_candidates) return CSD_ERR_NULL;
  const csd_shard_params& p = *pp;
  const int rc = shard_check(p);
  if (rc != CSD_OK) return rc;
  ShardArgs sa; StatsArgs st;
  shard_args(p, device_sms(nullptr), sa, st);
  sa.gathered = reinterpret_cast<const float4*>(records_all);
  sa.z_all = totals_all;
  sa.cand_local = out_candidates;
  const bool cfg = p.target_uncond != nullptr;
  cudaStream_t stream = (cudaStream_t)p.stream;
  if (p.dtype == CSD_F32) {
    if (cfg) shard_pick_kernel<float, true><<<p.B, kFinishThreads, 0, stream>>>(sa);
    else shard_pick_kernel<float, false><<<p.B, kFinishThreads, 0, stream>>>(sa);
  } else {
    if (cfg) shard_pick_kernel<__nv_bfloat16, true><<<p.B, kFinishThreads, 0, stream>>>(sa);
    else shard_pick_kernel<__nv_bfloat16, false><<<p.B, kFinishThreads, 0, stream>>>(sa);
  }
  return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

int csd_shard_emit(const csd_shard_params* pp, const int32_t* candidates_all, int32_t* out_tokens, int32_t* out_accept_len,
                   int32_t* out_status) {
  if (!pp || !candidates_all || !out_tokens || !out_accept_len) return CSD_ERR_NULL;
  const csd_shard_params& p = *pp;
  const int rc = shard_check(p);
  if (rc != CSD_OK) return rc;
  ShardArgs sa; StatsArgs st;
  shard_args(p, device_sms(nullptr), sa, st);
  sa.cand_all = candidates_all;
  sa.fin.out_tokens = out_tokens; sa.fin.out_accept_len = out_accept_len; sa.fin.out_status = out_status;
  shard_emit_kernel<<<p.B, 64, 0, (cudaStream_t)p.stream>>>(sa);
  return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

// ---- allocation-free form -------------------------------------------------------------
// Scratch that lives in the library's device image.  In host code the name below
// is only a handle for cudaGetSymbolAddress, never a device address: the kernels
// get the address that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[CSD_STATIC_SCRATCH_BYTES];

namespace {
void* g_static_scratch_addr[kMaxDevices];  // per device, filled on first use

// Device address of g_static_scratch on the current device; no allocation.
int static_scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CSD_ERR_LAUNCH;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return CSD_ERR_LAUNCH;
    }
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return CSD_OK;
}
}  // namespace

int csd_verify_static(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                      const float* uniforms, const float* relax_schedule, int B, int gamma, int V,
                      int32_t* out_tokens, int32_t* out_accept_len, void* stream) {
  if (!shape_ok(B, gamma, V)) return CSD_ERR_SHAPE;
  const size_t need = csd_workspace_size(B, gamma, V, CSD_F32);
  if (need > (size_t)CSD_STATIC_SCRATCH_BYTES) return CSD_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != CSD_OK) return rc;
  csd_params p;
  memset(&p, 0, sizeof p);
  p.target_logits = target_logits; p.draft_logits = draft_logits;
  p.cfg_scale = 1.0f; p.top_k = 0; p.dtype = CSD_F32;
  p.B = B; p.gamma = gamma; p.V = V; p.target_rows = gamma;
  p.draft_tokens = draft_tokens; p.uniforms = uniforms; p.relax_schedule = relax_schedule;
  p.out_tokens = out_tokens; p.out_accept_len = out_accept_len;
  p.workspace = scratch; p.workspace_bytes = CSD_STATIC_SCRATCH_BYTES;
  p.stream = stream;
  return verify_impl(p);
}

// ---- host-buffer form -----------------------------------------------------------
namespace {
struct HostPlan {
  size_t logits_t, logits_d, tokens, uniforms, schedule, out_tokens, out_len, out_status;
  size_t dbg_pqf, dbg_G;
  size_t off_t, off_d, off_tu, off_du, off_tok, off_uni, off_sched, off_otok, off_olen, off_ostat;
  size_t off_p, off_q, off_f, off_G, off_ws, ws_bytes, total;
  int64_t tstride, dstride;
};
bool host_plan(const csd_params& h, HostPlan& pl) {
  if (!shape_ok(h.B, h.gamma, h.V) || (h.dtype != CSD_F32 && h.dtype != CSD_BF16)) return false;
  if (h.target_rows != h.gamma && h.target_rows != h.gamma + 1) return false;
  pl.tstride = h.target_batch_stride ? h.target_batch_stride : (int64_t)h.target_rows * h.V;
  pl.dstride = h.draft_batch_stride ? h.draft_batch_stride : (int64_t)h.gamma * h.V;
  if (pl.tstride < (int64_t)h.target_rows * h.V || pl.dstride < (int64_t)h.gamma * h.V) return false;
  const size_t es = elem_size(h.dtype);
  pl.logits_t = (size_t)h.B * pl.tstride * es;
  pl.logits_d = (size_t)h.B * pl.dstride * es;
  pl.tokens = (size_t)h.B * h.gamma * 4;
  pl.uniforms = (size_t)h.B * (h.gamma + 1) * 4;
  pl.schedule = (size_t)h.gamma * 4;
  pl.out_tokens = (size_t)h.B * (h.gamma + 1) * 4;
  pl.out_len = (size_t)h.B * 4;
  pl.out_status = (size_t)h.B * 4;
  pl.dbg_pqf = (size_t)h.B * h.gamma * 4;
  pl.dbg_G = (size_t)h.B * h.V * 4;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  pl.off_t = take(pl.logits_t);
  pl.off_d = take(pl.logits_d);
  pl.off_tu = take(h.target_uncond ? pl.logits_t : 0);
  pl.off_du = take(h.draft_uncond ? pl.logits_d : 0);
  pl.off_tok = take(pl.tokens);
  pl.off_uni = take(pl.uniforms);
  pl.off_sched = take(pl.schedule);
  pl.off_otok = take(pl.out_tokens);
  pl.off_olen = take(pl.out_len);
  pl.off_ostat = take(pl.out_status);
  pl.off_p = take(h.dbg_p ? pl.dbg_pqf : 0);
  pl.off_q = take(h.dbg_q ? pl.dbg_pqf : 0);
  pl.off_f = take(h.dbg_f ? pl.dbg_pqf : 0);
  pl.off_G = take(h.dbg_G ? pl.dbg_G : 0);
  pl.ws_bytes = layout_for(h.B, h.gamma, h.V, h.dtype).total;
  pl.off_ws = take(pl.ws_bytes);
  pl.total = off;
  return true;
}
}  // namespace

size_t csd_host_staging_size(const csd_params* host) {
  HostPlan pl;
  if (!host || !host_plan(*host, pl)) return 0;
  return pl.total;
}

int csd_verify_host(const csd_params* host, void* staging, size_t staging_bytes) {
  if (!host) return CSD_ERR_NULL;
  const csd_params& h = *host;
  if (!h.target_logits || !h.draft_logits || !h.draft_tokens || !h.uniforms || !h.relax_schedule ||
      !h.out_tokens || !h.out_accept_len)
    return CSD_ERR_NULL;
  if (h.dtype != CSD_F32 && h.dtype != CSD_BF16) return CSD_ERR_DTYPE;
  if ((h.target_uncond == nullptr) != (h.draft_uncond == nullptr)) return CSD_ERR_ARG;
  HostPlan pl;
  if (!host_plan(h, pl)) return CSD_ERR_SHAPE;
  if (!staging || ((uintptr_t)staging % kAlign) != 0 || staging_bytes < pl.total) return CSD_ERR_WORKSPACE;
  char* base = (char*)staging;
  cudaStream_t stream = (cudaStream_t)h.stream;
  auto h2d = [&](size_t off, const void* src, size_t bytes) {
    return cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, stream);
  };
  auto d2h = [&](void* dst, size_t off, size_t bytes) {
    return cudaMemcpyAsync(dst, base + off, bytes, cudaMemcpyDeviceToHost, stream);
  };
  cudaError_t e = h2d(pl.off_t, h.target_logits, pl.logits_t);
  if (e == cudaSuccess) e = h2d(pl.off_d, h.draft_logits, pl.logits_d);
  if (e == cudaSuccess && h.target_uncond) e = h2d(pl.off_tu, h.target_uncond, pl.logits_t);
  if (e == cudaSuccess && h.draft_uncond) e = h2d(pl.off_du, h.draft_uncond, pl.logits_d);
  if (e == cudaSuccess) e = h2d(pl.off_tok, h.draft_tokens, pl.tokens);
  if (e == cudaSuccess) e = h2d(pl.off_uni, h.uniforms, pl.uniforms);
  if (e == cudaSuccess) e = h2d(pl.off_sched, h.relax_schedule, pl.schedule);
  if (e != cudaSuccess) return CSD_ERR_LAUNCH;

  csd_params d = h;
  d.target_logits = base + pl.off_t;
  d.draft_logits = base + pl.off_d;
  d.target_uncond = h.target_uncond ? base + pl.off_tu : nullptr;
  d.draft_uncond = h.draft_uncond ? base + pl.off_du : nullptr;
  d.target_batch_stride = pl.tstride;
  d.draft_batch_stride = pl.dstride;
  d.draft_tokens = (const int32_t*)(base + pl.off_tok);
  d.uniforms = (const float*)(base + pl.off_uni);
  d.relax_schedule = (const float*)(base + pl.off_sched);
  d.out_tokens = (int32_t*)(base + pl.off_otok);
  d.out_accept_len = (int32_t*)(base + pl.off_olen);
  d.out_status = (int32_t*)(base + pl.off_ostat);
  d.dbg_p = h.dbg_p ? (float*)(base + pl.off_p) : nullptr;
  d.dbg_q = h.dbg_q ? (float*)(base + pl.off_q) : nullptr;
  d.dbg_f = h.dbg_f ? (float*)(base + pl.off_f) : nullptr;
  d.dbg_G = h.dbg_G ? (float*)(base + pl.off_G) : nullptr;
  d.workspace = base + pl.off_ws;
  d.workspace_bytes = pl.ws_bytes;
  d.back_to_back = 0;   // the kernel follows its own input copies: ordinary stream order
  d.diag_accept_mass = nullptr;   // (device-only outputs: not part of the host form)
  d.diag_bound_term = nullptr;
  if (cudaMemsetAsync(d.workspace, 0, layout_for(h.B, h.gamma, h.V, h.dtype).zero_bytes, stream) != cudaSuccess)
    return CSD_ERR_LAUNCH;
  const int rc = verify_impl(d);
  if (rc != CSD_OK) return rc;

  e = d2h(h.out_tokens, pl.off_otok, pl.out_tokens);
  if (e == cudaSuccess) e = d2h(h.out_accept_len, pl.off_olen, pl.out_len);
  if (e == cudaSuccess && h.out_status) e = d2h(h.out_status, pl.off_ostat, pl.out_status);
  if (e == cudaSuccess && h.dbg_p) e = d2h(h.dbg_p, pl.off_p, pl.dbg_pqf);
  if (e == cudaSuccess && h.dbg_q) e = d2h(h.dbg_q, pl.off_q, pl.dbg_pqf);
  if (e == cudaSuccess && h.dbg_f) e = d2h(h.dbg_f, pl.off_f, pl.dbg_pqf);
  if (e == cudaSuccess && h.dbg_G) e = d2h(h.dbg_G, pl.off_G, pl.dbg_G);
  return e == cudaSuccess ? CSD_OK : CSD_ERR_LAUNCH;
}

// ---- schedules (host arithmetic, fp64, rounded once to fp32) -------------------------
int csd_make_schedule(int kind, double delta, double nu_or_ell, int L, float* out_host) {
  if (!out_host) return CSD_ERR_NULL;
  if (L < 1 || !(delta >= 0.0) || !isfinite(delta)) return CSD_ERR_ARG;
  if (kind == 0) {
    for (int i = 0; i < L; ++i) out_host[i] = (float)delta;
    return CSD_OK;
  }
  if (kind == 1) {
    const double nu = nu_or_ell;
    if (!(nu >= 0.0) || !isfinite(nu)) return CSD_ERR_ARG;
    // geometric weights exp(-nu (i-1)), normalised so that the multipliers average delta
    double norm = 0.0, w = 1.0;
    const double ratio = exp(-nu);
    for (int i = 0; i < L; ++i) { norm += w; w *= ratio; }
    w = delta * (double)L / norm;
    for (int i = 0; i < L; ++i) { out_host[i] = (float)w; w *= ratio; }
    return CSD_OK;
  }
  if (kind == 2) {
    const double ell = nu_or_ell;
    if (!(ell > 1.0) || !isfinite(ell)) return CSD_ERR_ARG;
    double norm = 0.0;
    for (int i = 1; i <= L; ++i) norm += fmax(0.0, ell - (double)i);
    if (!(norm > 0.0)) return CSD_ERR_ARG;
    for (int i = 1; i <= L; ++i) out_host[i - 1] = (float)(delta * (double)L * fmax(0.0, ell - (double)i) / norm);
    return CSD_OK;
  }
  return CSD_ERR_ARG;
}

const char* csd_error_string(int code) {
  switch (code) {
    case CSD_OK: return "ok";
    case CSD_ERR_NULL: return "a required pointer is NULL";
    case CSD_ERR_SHAPE: return "bad shape: need B >= 1, 1 <= gamma <= 32, 2 <= V <= 2^20, target_rows in {gamma, gamma+1}, strides covering the rows";
    case CSD_ERR_DTYPE: return "unknown dtype (CSD_F32 or CSD_BF16)";
    case CSD_ERR_WORKSPACE: return "workspace missing, not 256-byte aligned, or too small";
    case CSD_ERR_ARG: return "inconsistent or unsupported options";
    case CSD_ERR_LAUNCH: return "CUDA runtime error while enqueueing work";
    case CSD_ERR_ALIGN: return "csd_verify needs 16-byte aligned logits with V a multiple of 4 and at least 128; use csd_verify_ex with a workspace";
    case CSD_ERR_STATIC_LIMIT: return "problem too large for the built-in scratch of csd_verify_static (CSD_STATIC_SCRATCH_BYTES); use csd_verify_ex with a caller workspace";
    default: return "unknown error code";
  }
}

int csd_version(void) { return 400; }

}  // extern "C"
