// Tree-structured verification (the draft structure of the paper's experiments: a static tree of
// candidates; Algorithm 1 states the chain).  Reading of several candidates per node: they are
// independent draws from the drafter's distribution Q in the node's context, tried in stored order;
// with R the target's distribution there, a candidate x at level i is accepted with probability
// min{1, omega_i R(x)/Q(x)} (Eq. relax on the current residual); a rejection replaces R by
// Norm([R - Q f(.)]_+) (Eq. opt_G applied to R) and the next sibling is tried against that; when all
// are rejected the emitted token is drawn from the last residual, and a node without children ends
// the walk with a bonus token from the target's distribution.  A chain is Algorithm 1 itself.
//
// Contexts: 0 is the root, n + 1 the context after node n; row c of both logit arrays is the
// model's output in context c.  The row statistics of all 2 (N + 1) rows come from the kernels of
// csd_kernels.cuh (a call looks to them like a chain of N + 1 positions); tree_finish_kernel, one
// block per sequence, then walks the tree.  Every rejection costs one pass over the two rows of the
// current context (its normaliser Z).  The residual after k rejections is evaluated token by token
// by running the k-step recursion from the two logits; where two float[V] tables fit the block's shared
// memory, the residual and Q of the current context are kept there instead and updated in place.
#pragma once
#include "csd_kernels.cuh"

namespace csd {

constexpr int kMaxTreeNodes = 63;   // contexts: 64
constexpr int kMaxTreeDepth = 32;
constexpr int kMaxSiblings = 8;     // candidates of one node

struct TreeArgs {
  FinishArgs fin;        // gamma = T = N + 1 (contexts); tokens [B, N]; uniforms [B, N + 1]; schedule [D];
                         // out_tokens [B, D + 1]
  int N, D;
  int32_t* out_nodes;    // [B, D] or null
  int tab_off;           // > 0: the block's dynamic shared memory holds, at this offset (in doubles, after the tile
                         //      sums), two float[V] tables (see the kernel); 0: no room for them
  signed char parent[kMaxTreeNodes + 1];
};

struct TreeSmem {
  float M[2][kMaxTreeNodes + 1], S[2][kMaxTreeNodes + 1], thr[2][kMaxTreeNodes + 1];
  int valid[2][kMaxTreeNodes + 1];
  float inv_z[kMaxSiblings];   // 1 / Z_k of the rejections so far in the current context
  int keep[kMaxSiblings];      // the k-th update found an empty positive part and kept the residual
  int decision;                // thread 0's accept decision, for everybody
  FinishSmem pick;             // Z, tile and prefix of the draw
  int path_tok[kMaxTreeDepth + 1];
  int path_node[kMaxTreeDepth];
  // fetched for all nodes at once before the walk, so that its accept tests wait for no memory: every
  // node's token, that token's (filtered) logits in the two rows of its parent's context, its uniform
  int tok[kMaxTreeNodes];
  float tokz[2][kMaxTreeNodes];
  float uni[kMaxTreeNodes];
};

// Unnormalised residual after `k` rejections at one token: g_k(x), where g_1 = [P - min{Q, omega P}]_+
// (the cancellation-free form of weight_of), R_j = g_j / Z_j and g_{j+1} = [R_j - min{Q, omega R_j}]_+.
// k = 0 gives P itself.  With no usable drafter row (mode 1) every residual is P.
__device__ __forceinline__ float residual_of(float zt, float zd, const PairCtx& c, const float omega, const int k,
                                             const float* inv_z, const int* keep) {
  const float P = ex2f((zt - c.Mt) * kLog2e) * c.inv_t;
  if (k == 0 || c.mode == 1) return P;
  float g = keep[0] ? P : weight_of(zt, zd, c);
  if (k == 1) return g;
  const float Q = ex2f((zd - c.Md) * kLog2e) / (1.0f + c.Sd);
  for (int j = 1; j < k; ++j) {
    const float R = g * inv_z[j - 1];
    g = keep[j] ? R : fmaxf(0.0f, R - fminf(Q, omega * R));
  }
  return g;
}

template <typename T, bool CFG>
__global__ void __launch_bounds__(kFinishThreads, 1) tree_finish_kernel(const TreeArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  constexpr int NT = kFinishThreads;
  extern __shared__ double tile_sums[];   // one fp64 sum per tile
  __shared__ TreeSmem sm;
  pdl_wait();   // everything the statistics kernel wrote is visible from here on
  const FinishArgs& f = a.fin;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  const int N = a.N, C = N + 1, V = f.V, D = a.D;
  const int rows_per_seq = 2 * C;
  const int ntiles = (V + TILE - 1) / TILE;
  // Where they fit, two tables over the vocabulary live in shared memory while the walk stays in one
  // context: the current residual g_k(x) and the drafter's Q(x).  A rejection then updates the residual
  // in place (a few operations per token) instead of running the k-step recursion from the logits again;
  // the values are the same bits either way.
  float* const tabG = a.tab_off > 0 ? reinterpret_cast<float*>(tile_sums + a.tab_off) : nullptr;
  float* const tabQ = tabG ? tabG + V : nullptr;
  const T* tgt = reinterpret_cast<const T*>(f.target) + (int64_t)b * f.tstride;
  const T* dft = reinterpret_cast<const T*>(f.draft) + (int64_t)b * f.dstride;
  const T* tgt_u = CFG ? reinterpret_cast<const T*>(f.target_uncond) + (int64_t)b * f.tstride : nullptr;
  const T* dft_u = CFG ? reinterpret_cast<const T*>(f.draft_uncond) + (int64_t)b * f.dstride : nullptr;

  // ---- statistics of every context's two rows: merge the parts ------------------------------
  for (int r = warp; r < rows_per_seq; r += NT / 32) {
    const int which = r < C ? 0 : 1, c = r < C ? r : r - C;
    const int64_t row_id = (int64_t)b * rows_per_seq + r;
    float m = CSD_NEG_INF, s = -1.0f;
    for (int p = lane; p < f.parts; p += 32) {
      const float2 v = __ldcg(f.partials + row_id * f.parts + p);
      stat_merge(m, s, v.x, v.y);
    }
    stat_warp_allreduce(m, s);
    if (lane == 0) {
      sm.M[which][c] = m;
      sm.S[which][c] = s;
      sm.thr[which][c] = f.use_topk ? __ldcg(f.thresholds + row_id) : CSD_NEG_INF;
      sm.valid[which][c] = m > CSD_NEG_INF && m < CSD_POS_INF && s >= 0.0f && s < CSD_POS_INF;
    }
  }
  __syncthreads();

  if (tid < N) {
    const int n = tid, c = a.parent[n] + 1;
    const int tok = f.tokens[(int64_t)b * N + n];
    sm.tok[n] = tok;
    sm.uni[n] = f.uniforms[(int64_t)b * (N + 1) + n];
    float zt = 0.0f, zd = 0.0f;
    if (tok >= 0 && tok < V && sm.valid[0][c] && sm.valid[1][c]) {
      const Row<T, CFG> qt{tgt + (int64_t)c * V, CFG ? tgt_u + (int64_t)c * V : nullptr, f.cfg_scale, sm.thr[0][c] CSD_ROW_LEN(V)};
      const Row<T, CFG> qd{dft + (int64_t)c * V, CFG ? dft_u + (int64_t)c * V : nullptr, f.cfg_scale, sm.thr[1][c] CSD_ROW_LEN(V)};
      zt = qt.filter(qt.load_one(tok));
      zd = qd.filter(qd.load_one(tok));
    }
    sm.tokz[0][n] = zt;
    sm.tokz[1][n] = zd;
  }
  __syncthreads();

  // ---- the walk (every thread follows it; thread 0 takes the accept decisions) ---------------
  const float u = f.uniforms[(int64_t)b * (N + 1) + N];
  int status = 0, level = 0, ctx = 0, token = -1;
  int k = 0;                // rejections in the final context (depth of the residual drawn from)
  bool drew = false;
  PairCtx pc;
  Row<T, CFG> rt, rd;
  float omega = 0.0f;
  bool use_tab = false;   // the current context's residual and Q are tabulated (once it has had a rejection)
  for (;;) {
    const bool t_ok = sm.valid[0][ctx] != 0;
    rt = Row<T, CFG>{tgt + (int64_t)ctx * V, CFG ? tgt_u + (int64_t)ctx * V : nullptr, f.cfg_scale, sm.thr[0][ctx] CSD_ROW_LEN(V)};
    rd = Row<T, CFG>{dft + (int64_t)ctx * V, CFG ? dft_u + (int64_t)ctx * V : nullptr, f.cfg_scale, sm.thr[1][ctx] CSD_ROW_LEN(V)};
    pc.Mt = sm.M[0][ctx]; pc.St = sm.S[0][ctx];
    pc.inv_t = 1.0f / (1.0f + pc.St);
    int first_child = -1;
    for (int n = 0; n < N; ++n)
      if (a.parent[n] == ctx - 1) { first_child = n; break; }
    k = 0;
    if (first_child < 0 || level >= D) {   // a leaf: bonus token from the target's distribution here
      use_tab = false;
      pc.mode = 1; pc.Md = 0.0f; pc.Sd = 0.0f; pc.inv_den = pc.inv_t; pc.one_minus_omega = 1.0f;
      if (!t_ok) status |= 1;
      drew = t_ok;
      break;
    }
    const bool d_ok = sm.valid[1][ctx] != 0;
    pc.mode = d_ok ? 0 : 1;
    pc.Md = d_ok ? sm.M[1][ctx] : 0.0f; pc.Sd = d_ok ? sm.S[1][ctx] : 0.0f;
    pc.inv_den = pc.inv_t / (1.0f + pc.Sd);
    omega = f.schedule[level];
    omega = omega >= 0.0f ? omega : 0.0f;
    pc.one_minus_omega = 1.0f - omega;
    int accepted = -1;
    use_tab = tabG != nullptr && pc.mode == 0 && t_ok;   // (the same in every thread; tables are filled by this context's first rejection)
    for (int n = first_child; n < N; ++n) {
      if (a.parent[n] != ctx - 1) continue;
      // ---- accept test of candidate n against the residual after k rejections -------------------
      if (tid == 0) {
        const int tok = sm.tok[n];
        const bool tok_ok = tok >= 0 && tok < V;
        float fa = 0.0f;
        int flag = 0;
        if (!t_ok || !d_ok) flag = 1;
        else if (!tok_ok) flag = 2;
        else {
          const float zt = sm.tokz[0][n], zd = sm.tokz[1][n];
          const float dt = zt - pc.Mt, dd = zd - pc.Md;
          if (dd == CSD_NEG_INF) fa = 1.0f;            // q = 0: p/q = +inf, and 0/0 := 1
          else if (k == 0) {
            if (dt == CSD_NEG_INF) fa = 0.0f;          // p = 0 < q
            else fa = fminf(1.0f, omega * ex2f((dt - dd) * kLog2e) * ((1.0f + pc.Sd) / (1.0f + pc.St)));
          } else {
            const float R = (use_tab ? tabG[tok] : residual_of(zt, zd, pc, omega, k, sm.inv_z, sm.keep)) * sm.inv_z[k - 1];
            const float Q = ex2f(dd * kLog2e) / (1.0f + pc.Sd);
            fa = R > 0.0f ? fminf(1.0f, omega * R / Q) : 0.0f;
          }
        }
        const float r = sm.uni[n];
        sm.decision = ((r <= fa) ? 1 : 0) | (flag << 1);
      }
      __syncthreads();
      const int dec = sm.decision;
      __syncthreads();
      status |= dec >> 1;
      if (dec & 1) { accepted = n; break; }
      if (!t_ok) continue;   // nothing to update: the emitted token will be -1
      // ---- rejected: one pass for the normaliser of the next residual -----------------------------
      if (k >= kMaxSiblings) { status |= 4; continue; }   // (the host refuses such trees)
      if (tid == 0) sm.keep[k] = 0;
      __syncthreads();
      for (int attempt = 0; attempt < 2; ++attempt) {
        if (use_tab && k >= 1 && attempt == 1) {
          // the update found an empty positive part and has overwritten the table: bring g_k back from the logits
          for (int tile = warp; tile < ntiles; tile += NT / 32) {
            const int x0 = tile * TILE + lane * VEC;
            float zt[VEC], zd[VEC];
            rt.load_tile(x0, V, f.vec_ok, zt);
            rd.load_tile(x0, V, f.vec_ok, zd);
#pragma unroll
            for (int e = 0; e < VEC; ++e)
              if (x0 + e < V) tabG[x0 + e] = residual_of(rt.filter(zt[e]), rd.filter(zd[e]), pc, omega, k, sm.inv_z, sm.keep);
          }
          __syncthreads();
        }
        for (int tile = warp; tile < ntiles; tile += NT / 32) {
          const int x0 = tile * TILE + lane * VEC;
          float acc = 0.0f;
          if (use_tab && k >= 1) {
            // g_{k+1} from the tabulated g_k and Q: the last step of residual_of's recursion
            const float iz = sm.inv_z[k - 1];
            const bool kp = sm.keep[k] != 0;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              if (x0 + e < V) {
                const float R = tabG[x0 + e] * iz;
                const float gn = kp ? R : fmaxf(0.0f, R - fminf(tabQ[x0 + e], omega * R));
                tabG[x0 + e] = gn;
                acc += gn;
              }
            }
          } else {
            float zt[VEC], zd[VEC];
            rt.load_tile(x0, V, f.vec_ok, zt);
            if (pc.mode == 0) rd.load_tile(x0, V, f.vec_ok, zd);
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              const float ft = rt.filter(zt[e]), fd = pc.mode == 0 ? rd.filter(zd[e]) : 0.0f;
              const float gn = residual_of(ft, fd, pc, omega, k + 1, sm.inv_z, sm.keep);
              if (use_tab && x0 + e < V) {   // (k == 0: the tables are filled here)
                tabG[x0 + e] = gn;
                tabQ[x0 + e] = ex2f((fd - pc.Md) * kLog2e) / (1.0f + pc.Sd);
              }
              acc += gn;
            }
          }
          const double tsum = warp_sum_double((double)acc);
          if (lane == 0) tile_sums[tile] = tsum;
        }
        __syncthreads();
        if (warp == 0) locate_crossing_tile(tile_sums, ntiles, u, lane, sm.pick);
        __syncthreads();
        const double Z = sm.pick.Z;
        if ((Z > 0.0 && Z < (double)CSD_POS_INF) || attempt == 1) {
          if (tid == 0) sm.inv_z[k] = (Z > 0.0 && Z < (double)CSD_POS_INF) ? (float)(1.0 / Z) : 0.0f;
          break;
        }
        // empty positive part: the residual stays as it is
        status |= 4;
        if (tid == 0) sm.keep[k] = 1;
        __syncthreads();
      }
      __syncthreads();
      ++k;
    }
    if (accepted >= 0) {
      if (tid == 0) {
        sm.path_tok[level] = f.tokens[(int64_t)b * N + accepted];
        sm.path_node[level] = accepted;
      }
      ++level;
      ctx = accepted + 1;
      continue;
    }
    drew = t_ok && k > 0;
    break;
  }

  // ---- the draw: from the residual after k rejections (tile sums and tile are those of the last
  // pass), or, at a leaf, from the target's distribution ------------------------------------------
  double Z = 0.0;
  if (drew) {
    if (k == 0) {   // a leaf: no pass has run here yet
      for (int tile = warp; tile < ntiles; tile += NT / 32) {
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC];
        rt.load_tile(x0, V, f.vec_ok, zt);
        float acc = 0.0f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc += residual_of(rt.filter(zt[e]), 0.0f, pc, omega, 0, sm.inv_z, sm.keep);
        const double tsum = warp_sum_double((double)acc);
        if (lane == 0) tile_sums[tile] = tsum;
      }
      __syncthreads();
      if (warp == 0) locate_crossing_tile(tile_sums, ntiles, u, lane, sm.pick);
      __syncthreads();
    }
    Z = sm.pick.Z;
    if (Z > 0.0 && Z < (double)CSD_POS_INF) {
      if (warp == 0) {
        const int tile = sm.pick.pick_tile;
        int tok = -1;
        if (tile >= 0) {
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC], g[VEC];
          if (use_tab && k > 0) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) g[e] = x0 + e < V ? tabG[x0 + e] : 0.0f;
          } else {
            rt.load_tile(x0, V, f.vec_ok, zt);
            if (pc.mode == 0 && k > 0) rd.load_tile(x0, V, f.vec_ok, zd);
#pragma unroll
            for (int e = 0; e < VEC; ++e)
              g[e] = residual_of(rt.filter(zt[e]), (pc.mode == 0 && k > 0) ? rd.filter(zd[e]) : 0.0f, pc, omega, k, sm.inv_z, sm.keep);
          }
          tok = pick_in_tile<VEC>(g, x0, sm.pick.pick_prefix, (double)u * Z, lane);
        }
        if (lane == 0) sm.pick.token = tok;
      }
      __syncthreads();
      token = sm.pick.token;
    }
  }
  // ---- outputs ---------------------------------------------------------------------------------
  if (f.dbg_G) {
    float* G_out = f.dbg_G + (int64_t)b * V;
    if (token >= 0) {
      const float invZ = (float)(1.0 / Z);
      for (int tile = warp; tile < ntiles; tile += NT / 32) {
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC], zd[VEC];
        if (use_tab && k > 0) {
#pragma unroll
          for (int e = 0; e < VEC; ++e)
            if (x0 + e < V) G_out[x0 + e] = tabG[x0 + e] * invZ;
          continue;
        }
        rt.load_tile(x0, V, f.vec_ok, zt);
        if (pc.mode == 0 && k > 0) rd.load_tile(x0, V, f.vec_ok, zd);
#pragma unroll
        for (int e = 0; e < VEC; ++e)
          if (x0 + e < V)
            G_out[x0 + e] = residual_of(rt.filter(zt[e]), (pc.mode == 0 && k > 0) ? rd.filter(zd[e]) : 0.0f, pc, omega, k,
                                        sm.inv_z, sm.keep) * invZ;
      }
    } else {
      for (int x = tid; x < V; x += NT) G_out[x] = 0.0f;
    }
  }
  __syncthreads();
  if (tid <= D) {
    int v = -1;
    if (tid < level) v = sm.path_tok[tid];
    else if (tid == level) v = token;
    f.out_tokens[(int64_t)b * (D + 1) + tid] = v;
    if (a.out_nodes && tid < D) a.out_nodes[(int64_t)b * D + tid] = tid < level ? sm.path_node[tid] : -1;
  }
  if (tid == 0) {
    f.out_accept_len[b] = level;
    if (f.out_status) f.out_status[b] = status;
  }
}

}  // namespace csd
