// Vocabulary-sharded verification: every rank of a tensor-parallel LM head holds a contiguous slice
// [v_offset, v_offset + Vs) of every logit row.  One round of Algorithm 1 then needs three small
// exchanges between the ranks, and between them these kernels on each rank's own slice:
//
//   shard_merge_kernel    after row_stats_kernel on the slice: per row one record (m, s, logit of the
//                         drafted token if it lies in this slice, else -inf)
//        -- all-gather of the records --
//   shard_partial_kernel  one block per sequence: merges the ranks' records into the rows' global
//                         (m, s), runs the accept tests (Eq. relax) and finds tau -- every rank gets the
//                         same answer from the same numbers in the same order --, then sums Eq. opt_G
//                         at position tau + 1 over its own slice, per tile, with the GLOBAL statistics
//        -- all-gather of the slices' totals --
//   shard_pick_kernel     the slice that holds the crossing C(x) > u Z (totals of the slices before it
//                         give its starting value) picks the token; the others report none
//        -- all-gather of the candidates --
//   shard_emit_kernel     emits x_{1:tau+1} on every rank
//
// The inverse CDF runs in token-id order, so slices must be numbered in vocabulary order.  Top-k
// filtering needs the k-th largest value over all slices and is not part of this variant.
#pragma once
#include "csd_kernels.cuh"

namespace csd {

struct ShardArgs {
  FinishArgs fin;          // this rank's slice: V = Vs, strides of the slice arrays; parts/partials of row_stats_kernel
  int n_shards, shard;     // ranks, and this rank's index in vocabulary order
  int v_offset;            // global id of the slice's first token
  int V_total;
  float4* local;           // [rows] out of shard_merge_kernel: (m, s, token logit, 0)
  const float4* gathered;  // [n_shards][rows]
  double* tile_sums;       // workspace: [B][ntiles] of this slice
  float4* ctx;             // workspace: [B][4] what the draw of a sequence needs, kept between the calls
  double* z_local;         // [B][2]: this slice's total of Eq. opt_G at the draw position, and of P there
  const double* z_all;     // [n_shards][B][2]
  int32_t* cand_local;     // [B][2]: token picked in this slice (global id) or -1; status bits
  const int32_t* cand_all; // [n_shards][B][2]
};

// ---- step 1b: one record per row of the slice ------------------------------------------------------
template <typename T, bool CFG>
__global__ void __launch_bounds__(256) shard_merge_kernel(const ShardArgs a) {
  const FinishArgs& f = a.fin;
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rows_per_seq = f.T + f.gamma;
  const int n_rows = f.B * rows_per_seq;
  const int row_id = blockIdx.x * 8 + warp;
  if (row_id >= n_rows) return;
  float m = CSD_NEG_INF, s = -1.0f;
  for (int p = lane; p < f.parts; p += 32) {
    const float2 v = __ldcg(f.partials + (int64_t)row_id * f.parts + p);
    stat_merge(m, s, v.x, v.y);
  }
  stat_warp_allreduce(m, s);
  if (lane == 0) {
    const int b = row_id / rows_per_seq, r = row_id - b * rows_per_seq;
    const int which = r < f.T ? 0 : 1, i = r < f.T ? r : r - f.T;
    float tokz = CSD_NEG_INF;
    if (i < f.gamma) {
      const int loc = f.tokens[(int64_t)b * f.gamma + i] - a.v_offset;
      if (loc >= 0 && loc < f.V) {
        const T* base = reinterpret_cast<const T*>(which == 0 ? f.target : f.draft);
        const T* ubase = CFG ? reinterpret_cast<const T*>(which == 0 ? f.target_uncond : f.draft_uncond) : nullptr;
        const int64_t off = (int64_t)b * (which == 0 ? f.tstride : f.dstride) + (int64_t)i * f.V;
        Row<T, CFG> row{base + off, CFG ? ubase + off : nullptr, f.cfg_scale, CSD_NEG_INF CSD_ROW_LEN(f.V)};
        tokz = row.load_one(loc);
      }
    }
    a.local[row_id] = make_float4(m, s, tokz, 0.0f);
  }
}

struct ShardSmem {
  float M[2][kMaxGamma + 1], S[2][kMaxGamma + 1], tokz[2][kMaxGamma + 1];
  int valid[2][kMaxGamma + 1];
  int acc[kMaxGamma], flag[kMaxGamma];
  FinishSmem pick;
};

// Global statistics of the rows of sequence b from all ranks' records; accept tests; returns tau and
// the status bits of the positions looked at.  Every rank computes this identically.
__device__ __forceinline__ int shard_accept(const ShardArgs& a, const int b, ShardSmem& sm, const int tid, int& status,
                                            float* dbg_row /* p, q, f of thread's position or null */) {
  const FinishArgs& f = a.fin;
  const int L = f.gamma, rows_per_seq = f.T + L, n_rows = f.B * rows_per_seq;
  const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  for (int r = warp; r < rows_per_seq; r += nwarps) {
    const int which = r < f.T ? 0 : 1, i = r < f.T ? r : r - f.T;
    float m = CSD_NEG_INF, s = -1.0f, tz = CSD_NEG_INF;
    for (int k = lane; k < a.n_shards; k += 32) {
      const float4 v = __ldcg(a.gathered + (int64_t)k * n_rows + (int64_t)b * rows_per_seq + r);
      stat_merge(m, s, v.x, v.y);
      tz = fmaxf(tz, v.z);
    }
    stat_warp_allreduce(m, s);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tz = fmaxf(tz, __shfl_xor_sync(0xffffffffu, tz, off));
    if (lane == 0) {
      sm.M[which][i] = m; sm.S[which][i] = s; sm.tokz[which][i] = tz;
      sm.valid[which][i] = m > CSD_NEG_INF && m < CSD_POS_INF && s >= 0.0f && s < CSD_POS_INF;
    }
  }
  __syncthreads();
  if (tid < L) {
    const int i = tid;
    const bool t_ok = sm.valid[0][i], d_ok = sm.valid[1][i];
    const int tok = f.tokens[(int64_t)b * L + i];
    const bool tok_ok = tok >= 0 && tok < a.V_total;
    float omega = f.schedule[i];
    omega = omega >= 0.0f ? omega : 0.0f;
    float fa = 0.0f, p = __int_as_float(0x7fc00000), q = p;
    int flag = 0;
    if (!t_ok || !d_ok) flag = 1;
    else if (!tok_ok) flag = 2;
    else {
      const float dt = sm.tokz[0][i] - sm.M[0][i], dd = sm.tokz[1][i] - sm.M[1][i];
      p = ex2f(dt * kLog2e) / (1.0f + sm.S[0][i]);
      q = ex2f(dd * kLog2e) / (1.0f + sm.S[1][i]);
      if (dd == CSD_NEG_INF) fa = 1.0f;         // q = 0: p/q = +inf, and 0/0 := 1
      else if (dt == CSD_NEG_INF) fa = 0.0f;    // p = 0 < q
      else fa = fminf(1.0f, omega * ex2f((dt - dd) * kLog2e) * ((1.0f + sm.S[1][i]) / (1.0f + sm.S[0][i])));
    }
    sm.acc[i] = (f.uniforms[(int64_t)b * (L + 1) + i] <= fa) ? 1 : 0;
    sm.flag[i] = flag;
    if (dbg_row) { dbg_row[0] = p; dbg_row[1] = q; dbg_row[2] = fa; }
  }
  __syncthreads();
  int tau = 0;
  while (tau < L && sm.acc[tau]) ++tau;
  status = 0;
  for (int i = 0; i <= min(tau, L - 1); ++i) status |= sm.flag[i];
  return tau;
}

// What the draw of one sequence needs, kept in the workspace between shard_partial_kernel and
// shard_pick_kernel: four float4.
struct ShardDraw {
  float Mt, St, Md, Sd;
  float one_minus_omega, u;
  int j, mode;      // row index of the draw (gamma: the bonus row); 0 Eq. opt_G, 1 from P, -1 nothing to draw from
  int tau, status;
  int pad[6];
};
static_assert(sizeof(ShardDraw) == 64, "four float4 per sequence");

template <typename T, bool CFG>
__device__ __forceinline__ void shard_rows(const FinishArgs& f, int b, int j, Row<T, CFG>& rt, Row<T, CFG>& rd) {
  const int jt = min(j, f.T - 1);
  const int64_t toff = (int64_t)b * f.tstride + (int64_t)jt * f.V;
  rt = Row<T, CFG>{reinterpret_cast<const T*>(f.target) + toff,
                   CFG ? reinterpret_cast<const T*>(f.target_uncond) + toff : nullptr, f.cfg_scale, CSD_NEG_INF CSD_ROW_LEN(f.V)};
  rd = rt;
  if (j < f.gamma) {
    const int64_t doff = (int64_t)b * f.dstride + (int64_t)j * f.V;
    rd = Row<T, CFG>{reinterpret_cast<const T*>(f.draft) + doff,
                     CFG ? reinterpret_cast<const T*>(f.draft_uncond) + doff : nullptr, f.cfg_scale, CSD_NEG_INF CSD_ROW_LEN(f.V)};
  }
}

// Per-tile sums of the draw's weights over this slice (mode 0: Eq. opt_G; mode 1: P), fp64 per tile.
template <typename T, bool CFG>
__device__ __forceinline__ void shard_tile_sums(const FinishArgs& f, const Row<T, CFG>& rt, const Row<T, CFG>& rd,
                                                const PairCtx& pc, double* tiles, const int tid) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int ntiles = (f.V + TILE - 1) / TILE;
  for (int tile = warp; tile < ntiles; tile += nwarps) {
    const int x0 = tile * TILE + lane * VEC;
    float zt[VEC], zd[VEC];
    rt.load_tile(x0, f.V, f.vec_ok, zt);
    if (pc.mode == 0) rd.load_tile(x0, f.V, f.vec_ok, zd);
    float acc = 0.0f;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc += weight_of(zt[e], pc.mode == 0 ? zd[e] : 0.0f, pc);
    const double tsum = warp_sum_double((double)acc);
    if (lane == 0) tiles[tile] = tsum;
  }
}

// ---- step 2: accept tests (replicated), tau, this slice's share of the draw's normaliser ------------
template <typename T, bool CFG>
__global__ void __launch_bounds__(kFinishThreads, 1) shard_partial_kernel(const ShardArgs a) {
  __shared__ ShardSmem sm;
  const FinishArgs& f = a.fin;
  constexpr int TILE = 32 * Elem<T>::kVec;
  const int tid = threadIdx.x, b = blockIdx.x, L = f.gamma;
  const int ntiles = (f.V + TILE - 1) / TILE;
  float pqf[3];
  int status;
  const int tau = shard_accept(a, b, sm, tid, status, (f.dbg_p || f.dbg_q || f.dbg_f) ? pqf : nullptr);
  if (tid < L && a.shard == 0) {   // (the same on every rank: one writes)
    if (f.dbg_p) f.dbg_p[(int64_t)b * L + tid] = pqf[0];
    if (f.dbg_q) f.dbg_q[(int64_t)b * L + tid] = pqf[1];
    if (f.dbg_f) f.dbg_f[(int64_t)b * L + tid] = pqf[2];
  }
  // which distribution the token comes from
  const int j = tau;
  int mode;
  if (j < L) mode = !sm.valid[0][j] ? -1 : (sm.valid[1][j] ? 0 : 1);
  else if (f.T == L + 1) { mode = sm.valid[0][L] ? 1 : -1; if (mode < 0) status |= 1; }
  else mode = -1;
  PairCtx pc;
  pc.Mt = sm.M[0][min(j, f.T - 1)]; pc.St = sm.S[0][min(j, f.T - 1)];
  pc.Md = j < L ? sm.M[1][j] : 0.0f; pc.Sd = j < L ? sm.S[1][j] : 0.0f;
  pc.inv_t = 1.0f / (1.0f + pc.St);
  pc.inv_den = pc.inv_t / (1.0f + pc.Sd);
  float omega = j < L ? f.schedule[j] : 0.0f;
  omega = omega >= 0.0f ? omega : 0.0f;
  pc.one_minus_omega = 1.0f - omega;
  pc.mode = mode == 0 ? 0 : 1;
  double* tiles = a.tile_sums + (int64_t)b * ntiles;
  double z_g = 0.0;
  if (mode >= 0) {
    Row<T, CFG> rt, rd;
    shard_rows<T, CFG>(f, b, j, rt, rd);
    shard_tile_sums<T, CFG>(f, rt, rd, pc, tiles, tid);
    __syncthreads();
    if (tid < 32) {   // the slice's total, in a fixed order
      double local = 0.0;
      for (int t = tid; t < ntiles; t += 32) local += tiles[t];
      z_g = warp_sum_double(local);
    }
  }
  if (tid == 0) {
    // this slice's share of the target distribution's mass at the draw row: what the fall-back needs
    // (Z of Eq. opt_G empty), known from the records without another pass
    const float4 mine = __ldcg(a.gathered + (int64_t)a.shard * f.B * (f.T + L) + (int64_t)b * (f.T + L) + min(j, f.T - 1));
    const double z_p = (mode >= 0 && mine.x > CSD_NEG_INF)
                           ? (double)((1.0f + mine.y) * ex2f((mine.x - pc.Mt) * kLog2e) * pc.inv_t) : 0.0;
    a.z_local[2 * b] = mode == 0 ? z_g : (mode == 1 ? z_g : 0.0);
    a.z_local[2 * b + 1] = z_p;
    ShardDraw d;
    d.Mt = pc.Mt; d.St = pc.St; d.Md = pc.Md; d.Sd = pc.Sd;
    d.one_minus_omega = pc.one_minus_omega;
    d.u = f.uniforms[(int64_t)b * (L + 1) + L];
    d.j = j; d.mode = mode; d.tau = tau; d.status = status;
    for (int k = 0; k < 6; ++k) d.pad[k] = 0;
    const float4* src = reinterpret_cast<const float4*>(&d);
    for (int k = 0; k < 4; ++k) a.ctx[4 * b + k] = src[k];
  }
}

// ---- step 3: the slice that holds the crossing picks the token ------------------------------------------
template <typename T, bool CFG>
__global__ void __launch_bounds__(kFinishThreads, 1) shard_pick_kernel(const ShardArgs a) {
  __shared__ FinishSmem sm;
  __shared__ double sh_target, sh_pre;
  __shared__ int sh_owner, sh_fallback;
  const FinishArgs& f = a.fin;
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  const int tid = threadIdx.x, lane = tid & 31, b = blockIdx.x;
  const int ntiles = (f.V + TILE - 1) / TILE;
  ShardDraw d;
  {
    float4* dst = reinterpret_cast<float4*>(&d);
    for (int k = 0; k < 4; ++k) dst[k] = a.ctx[4 * b + k];
  }
  int status = d.status, token = -1;
  if (d.mode >= 0) {
    PairCtx pc;
    pc.Mt = d.Mt; pc.St = d.St; pc.Md = d.Md; pc.Sd = d.Sd;
    pc.inv_t = 1.0f / (1.0f + pc.St);
    pc.inv_den = pc.inv_t / (1.0f + pc.Sd);
    pc.one_minus_omega = d.one_minus_omega;
    pc.mode = d.mode == 0 ? 0 : 1;
    if (tid == 0) {
      // totals of all slices, in vocabulary order; an empty positive part falls back to P_j
      double Z = 0.0;
      for (int k = 0; k < a.n_shards; ++k) Z += a.z_all[((int64_t)k * f.B + b) * 2];
      int which = 0;
      if (d.mode == 0 && !(Z > 0.0 && Z < (double)CSD_POS_INF)) {
        which = 1;
        Z = 0.0;
        for (int k = 0; k < a.n_shards; ++k) Z += a.z_all[((int64_t)k * f.B + b) * 2 + 1];
      }
      const double target = (double)d.u * Z;
      // the first slice whose running total passes the target owns the token; if none does (u >= 1,
      // rounding), the last slice with weight
      double c = 0.0, pre = 0.0;
      int owner = -1, last = -1;
      double pre_last = 0.0;
      for (int k = 0; k < a.n_shards; ++k) {
        const double zk = a.z_all[((int64_t)k * f.B + b) * 2 + which];
        if (zk > 0.0) { last = k; pre_last = c; }
        if (owner < 0 && zk > 0.0 && c + zk > target) { owner = k; pre = c; }
        c += zk;
      }
      if (owner < 0) { owner = last; pre = pre_last; }
      if (!(Z > 0.0 && Z < (double)CSD_POS_INF)) owner = -1;
      sh_owner = owner; sh_pre = pre; sh_target = target; sh_fallback = which;
    }
    __syncthreads();
    if (sh_fallback) { status |= 4; pc.mode = 1; }
    if (sh_owner == a.shard) {
      Row<T, CFG> rt, rd;
      shard_rows<T, CFG>(f, b, d.j, rt, rd);
      double* tiles = a.tile_sums + (int64_t)b * ntiles;
      if (sh_fallback) {   // the stored sums are those of Eq. opt_G: sum P over the slice instead
        shard_tile_sums<T, CFG>(f, rt, rd, pc, tiles, tid);
        __syncthreads();
      }
      const double target_local = sh_target - sh_pre;
      if (tid < 32) locate_crossing_tile(tiles, ntiles, d.u, lane, sm, &target_local);
      __syncthreads();
      if (tid < 32) {
        const int tile = sm.pick_tile;
        int tok = -1;
        if (tile >= 0) {
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC], g[VEC];
          rt.load_tile(x0, f.V, f.vec_ok, zt);
          if (pc.mode == 0) rd.load_tile(x0, f.V, f.vec_ok, zd);
#pragma unroll
          for (int e = 0; e < VEC; ++e) g[e] = weight_of(zt[e], pc.mode == 0 ? zd[e] : 0.0f, pc);
          tok = pick_in_tile<VEC>(g, x0, sm.pick_prefix, target_local, lane);
        }
        if (lane == 0) sm.token = tok;
      }
      __syncthreads();
      token = sm.token >= 0 ? sm.token + a.v_offset : -1;
    }
  }
  if (tid == 0) {
    a.cand_local[2 * b] = token;
    a.cand_local[2 * b + 1] = status;
  }
}

// ---- step 4: emit x_{1:tau+1} --------------------------------------------------------------------------
__global__ void shard_emit_kernel(const ShardArgs a) {
  const FinishArgs& f = a.fin;
  const int b = blockIdx.x, tid = threadIdx.x, L = f.gamma;
  __shared__ int sh_tok, sh_status;
  if (tid == 0) {
    int tok = -1, status = 0;
    for (int k = 0; k < a.n_shards; ++k) {
      tok = max(tok, a.cand_all[((int64_t)k * f.B + b) * 2]);
      status |= a.cand_all[((int64_t)k * f.B + b) * 2 + 1];
    }
    sh_tok = tok; sh_status = status;
  }
  __syncthreads();
  const ShardDraw* d = reinterpret_cast<const ShardDraw*>(a.ctx + 4 * b);
  const int tau = d->tau;
  if (tid <= L) {
    int v = -1;
    if (tid < tau) v = f.tokens[(int64_t)b * L + tid];
    else if (tid == tau) v = sh_tok;
    f.out_tokens[(int64_t)b * (L + 1) + tid] = v;
  }
  if (tid == 0) {
    f.out_accept_len[b] = tau;
    if (f.out_status) f.out_status[b] = sh_status;
  }
}

}  // namespace csd
