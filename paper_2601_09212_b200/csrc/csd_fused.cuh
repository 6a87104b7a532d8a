// Single-launch path of libcsd (sm_100a): one persistent kernel per call.
//
// Phase 1 streams this block's share of the logit rows through rings of
// shared-memory stages filled by bulk asynchronous copies (mbarrier completion)
// and keeps the per-row results in shared memory.  Phase 2 is the finish.  A block
// owns, for its sequence(s), a range of draft positions with both rows of each, so
// it runs the accept tests of its positions itself (Eq. relax).  Where a sequence is
// split over several blocks, these form one thread-block cluster: each stores what it
// found into its peers' shared memory, one cluster barrier later all of them know
// which block holds the first rejection, and that block alone draws the replacement
// token (Eq. opt_G with the two rows brought back through the ring, inverse CDF) and
// emits the sequence.  Every wait on a copy is bounded.
//
// Consecutive calls on a stream overlap (programmatic dependent launch): every block
// signals launch_dependents at once, and everything up to a block's first global write
// -- streaming, accept tests, the exchange, the draw -- reads only the call's inputs, so
// it runs beside the previous call; griddepcontrol.wait comes just before that first
// write, which keeps the outputs of consecutive calls in order.
//
//   verify_plain_kernel  every warp streams its own parts of rows through its own
//                        ring and keeps a running (m, s) per lane.
//   verify_topk_kernel   a block streams whole rows; the first stage of a row is
//                        the sample for a mean/deviation guess `lo` of a value a
//                        little below the k-th largest; values >= lo are gathered
//                        as they stream by; one histogram over them finds the bin
//                        of the k-th largest and an exact rank among that bin's
//                        few values gives the threshold.  When the guess does not
//                        bracket the answer the row is re-read from global memory
//                        and selected exactly by radix, so the result never
//                        depends on the guess.
#pragma once
#include <type_traits>

#include "csd_kernels.cuh"

namespace csd {

constexpr int kPlainThreads = 256;   // plain kernel: 8 independent warp pipelines, three blocks per SM
constexpr int kPlainWarps = kPlainThreads / 32;
constexpr int kTopkThreads = 256;    // top-k kernel: 8 warps per row, four blocks per SM
constexpr int kTopkWarps = kTopkThreads / 32;
constexpr long long kWaitCycles = 1ll << 31;  // about a second: then give up and flag it
constexpr int kFinTiles = 1024;               // tiles of 32 lanes x 16 bytes: V <= 131072 (fp32) / 262144 (bf16)

// ---- mbarrier and bulk-copy primitives -----------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  // the last operand is a hint: the hardware may park the thread for up to that many ns
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity), "r"(2000u)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within about `limit` cycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const long long limit = kWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// global -> shared bulk copy of `bytes` (multiple of 16; both addresses 16-byte aligned),
// completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}
// the same for `bytes` of a logit row of V elements starting at element x0; the checked build tests the
// range first and leaves a bad copy out (its wait then runs into the limit and reports TIMEOUT)
template <typename T>
__device__ __forceinline__ void bulk_load_row(void* dst, const T* row, int x0, uint32_t bytes, int V, uint64_t* bar) {
#ifdef CSD_CHECKED
  if (!checked_ok(x0, (int)(bytes / sizeof(T)), V, 3)) return;
#endif
  bulk_load(dst, row + x0, bytes, bar);
}
// orders this thread's earlier shared-memory accesses before a bulk copy it issues next
__device__ __forceinline__ void fence_before_bulk() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// maximum that returns NaN when either operand is NaN (fmaxf would drop it)
__device__ __forceinline__ float max_nan(float x, float y) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y));
  return r;
}

// ---- thread-block cluster: the blocks of one sequence ---------------------------------------
// Hardware barrier over all threads of all blocks of the cluster, split in two halves.  Every
// thread of every block executes each half the same number of times, in the same order.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// 32-bit store into the shared memory of block `rank` of this cluster, at the address that
// `local` has in this block
__device__ __forceinline__ void cluster_store(void* local, uint32_t rank, uint32_t v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr(local)), "r"(rank));
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"(v) : "memory");
}
// the same for a double
__device__ __forceinline__ void cluster_store_f64(void* local, uint32_t rank, double v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr(local)), "r"(rank));
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(remote), "d"(v) : "memory");
}
constexpr int kMaxCluster = 8;   // portable cluster size

template <typename T>
__device__ __forceinline__ void unpack_vec(const unsigned char* p, float (&out)[Elem<T>::kVec]);
template <>
__device__ __forceinline__ void unpack_vec<float>(const unsigned char* p, float (&out)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void unpack_vec<__nv_bfloat16>(const unsigned char* p, float (&out)[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    out[2 * k] = __uint_as_float(w[k] << 16);
    out[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
  }
}
template <typename T>
__device__ __forceinline__ float load_scalar_smem(const unsigned char* p);
template <>
__device__ __forceinline__ float load_scalar_smem<float>(const unsigned char* p) {
  return *reinterpret_cast<const float*>(p);
}
template <>
__device__ __forceinline__ float load_scalar_smem<__nv_bfloat16>(const unsigned char* p) {
  return __uint_as_float(((uint32_t) * reinterpret_cast<const unsigned short*>(p)) << 16);
}

// What a block found at the position it drew a token for.
struct alignas(16) SeqRecord {
  int first_rej;   // 0-based position of this block's first rejection, -1 if it accepted all of its positions
  int token;       // token drawn at first_rej; for the block that owns the bonus row and accepted everything,
                   // the bonus token; -1 if there was nothing to draw from
  int status_at;   // status bits of that draw (bad row, bad token, Z fallback; for the bonus draw: bad row)
  int status_any;  // status bits that hold wherever the sequence ends (a bounded wait gave up)
  int mode;        // diagnostics: how the token was drawn (0: Eq. opt_G, 1: from P), and the statistics used
  float Mt, St, Md, Sd, thr_t, thr_d, one_minus_omega;
  double Z;
  int pad[2];
};

struct FusedArgs {
  FinishArgs fin;       // inputs and outputs (the workspace arrays of the multi-launch path are unused)
  int chunks_per_part;  // plain kernel: warp stages per part
  int parts_per_row;    // plain kernel
  int ctas_per_seq;     // > 1: a sequence's positions are split over the blocks of one cluster of this
                        //      size; 1: a block owns seqs_per_cta whole sequences (no clusters)
  int seqs_per_cta;
  int top_k;
  float lo_sigmas;      // top-k guess: lo = mean + lo_sigmas * deviation (NaN: always select exactly)
  float lo_delta;       // how many deviations below a row's exact threshold the next guess should sit (< 0)
  float hi_delta;       // a level this many deviations above lo has, almost surely, fewer than k values above it
                        // (NaN: never take the short cut that needs it)
  int* error_flag;      // set when a bounded wait gave up; null: nobody asked for the status
  long long wait_limit; // cycles a wait on a copy may take (kWaitCycles unless a test shortens it)
  int large_lists;      // top-k: the instance with the large candidate lists (set by the host from k and V)
  float2* stats_out;    // not null: stop after the streaming phase and write every local row's (m, s) here,
  float* thr_out;       //   and its top-k threshold there (may be null), at row b * (T + gamma) + (target ? i : T + i)
  int drop_first_copy;  // test aid: the first copy of block 0 is announced to its barrier but never issued,
                        // so that the wait on it runs out (nothing is left in flight)
};

// ---- a block's share of the work ------------------------------------------------------
// Blocks are aligned with sequences AND with positions: a block owns, for each of its
// sequences, a range of draft positions and BOTH rows (target, drafter) of each, so that it can
// run the accept tests of its positions by itself and, if the sequence's first rejection turns out
// to be among them, draw the replacement token.  Local rows are ordered t_p0, d_p0, t_p0+1, d_p0+1,
// ..., [bonus row].
struct BlockShare {
  int seq_begin, seq_end;   // sequences this block works on
  int pos_begin, pos_end;   // draft positions (0-based) it owns of each
  int bonus;                // it also owns the bonus row (target row gamma)
  int rows_per_seq;         // local rows per sequence
  int n_rows;               // local rows in all
  int slot;                 // its rank among the blocks of the sequence (ctas_per_seq > 1)
};
__device__ __forceinline__ BlockShare block_share(const FusedArgs& a) {
  BlockShare sh;
  const int L = a.fin.gamma;
  const bool has_bonus_row = a.fin.T == L + 1;
  if (a.ctas_per_seq > 1) {
    const int b = blockIdx.x / a.ctas_per_seq;
    const int j = blockIdx.x - b * a.ctas_per_seq;
    sh.seq_begin = b;
    sh.seq_end = b + 1;
    sh.pos_begin = L * j / a.ctas_per_seq;
    sh.pos_end = L * (j + 1) / a.ctas_per_seq;
    sh.bonus = (has_bonus_row && j == a.ctas_per_seq - 1) ? 1 : 0;
    sh.slot = j;
  } else {
    sh.seq_begin = min(a.fin.B, (int)blockIdx.x * a.seqs_per_cta);
    sh.seq_end = min(a.fin.B, sh.seq_begin + a.seqs_per_cta);
    sh.pos_begin = 0;
    sh.pos_end = L;
    sh.bonus = has_bonus_row ? 1 : 0;
    sh.slot = 0;
  }
  sh.rows_per_seq = 2 * (sh.pos_end - sh.pos_begin) + sh.bonus;
  sh.n_rows = (sh.seq_end - sh.seq_begin) * sh.rows_per_seq;
  return sh;
}
// local row -> (sequence, 0 target / 1 drafter, position)
__device__ __forceinline__ void local_row(const BlockShare& sh, int r_loc, int gamma, int& b, int& which, int& i) {
  const int sl = r_loc < sh.rows_per_seq ? 0 : r_loc / sh.rows_per_seq;   // (usually one sequence: no division)
  const int r = r_loc - sl * sh.rows_per_seq;
  b = sh.seq_begin + sl;
  if (r < 2 * (sh.pos_end - sh.pos_begin)) { i = sh.pos_begin + (r >> 1); which = r & 1; }
  else { i = gamma; which = 0; }
}
template <typename T, bool CFG>
__device__ __forceinline__ Row<T, CFG> row_at(const FinishArgs& f, int b, int which, int i) {
  Row<T, CFG> row;
  row.scale = f.cfg_scale;
  row.thr = CSD_NEG_INF;
#ifdef CSD_CHECKED
  row.n = f.V;
#endif
  if (which == 0) {
    const int64_t off = (int64_t)b * f.tstride + (int64_t)i * f.V;
    row.cond = reinterpret_cast<const T*>(f.target) + off;
    row.uncond = CFG ? reinterpret_cast<const T*>(f.target_uncond) + off : nullptr;
  } else {
    const int64_t off = (int64_t)b * f.dstride + (int64_t)i * f.V;
    row.cond = reinterpret_cast<const T*>(f.draft) + off;
    row.uncond = CFG ? reinterpret_cast<const T*>(f.draft_uncond) + off : nullptr;
  }
  return row;
}
constexpr int kBlockRows = 128;   // local rows a block may own (the host keeps it within this; a tree's 64 contexts
                                  // are 128 rows)

// Per-row results of phase 1, in shared memory until the block's own finish consumes them.
struct RowStats {
  float2 ms[kBlockRows];     // (m, s) of the whole row
  float thr[kBlockRows];     // top-k threshold (-inf without top-k)
  float tokz[kBlockRows];    // logit of the row's drafted token (undefined for a bonus row or a token out of range);
                             // -inf if the top-k filter is known to drop it
};

// The logit of every local row's drafted token, by scalar loads straight from global memory (mixed like
// the rows), when the kernel starts: the loads are long complete when the row's statistics are.
template <typename T, bool CFG, int NT>
__device__ __forceinline__ void load_token_logits(const FinishArgs& f, const BlockShare& sh, const int tid, RowStats& rs) {
  for (int r = tid; r < sh.n_rows && r < kBlockRows; r += NT) {
    int b, which, i;
    local_row(sh, r, f.gamma, b, which, i);
    if (i >= f.gamma) continue;   // the bonus row has no drafted token
    const int tok = f.tokens[(int64_t)b * f.gamma + i];
    if (tok >= 0 && tok < f.V) rs.tokz[r] = row_at<T, CFG>(f, b, which, i).load_one(tok);
  }
}

// ---- the block's finish on its own positions ----------------------------------------------
struct FinishStage {
  int tok[kMaxGamma + 1];
  float uni[kMaxGamma + 1];
  float omega[kMaxGamma];
  float tokz[2][kMaxGamma + 1];
  float p[kMaxGamma], q[kMaxGamma], f[kMaxGamma];
  float mon_am[kMaxGamma], mon_bt[kMaxGamma];   // per-position monitors of Theorem 2, until they are written out
  SeqRecord rec;
  uint32_t xch[kMaxCluster];   // written by the blocks of the cluster: what each found (see finish_block)
  uint32_t share[kMaxCluster][12];   // written by every block of the cluster into every block, together with xch:
                                     // what the draw's weights need if that block turns out to hold the
                                     // sequence's first rejection (see finish_block, cluster_draw)
  alignas(8) uint64_t bar;
  alignas(8) uint64_t bar2;    // second copy barrier of the per-position monitors
};

// Eq. opt_G summed per tile over the whole row pair, rows brought through the ring by bulk copies;
// then the tile of the crossing and the token inside it.  Returns the token (-1: nothing to draw
// from); Z_out gets the normaliser, status gets bits 4 / 8 where they apply; ctx.mode may change to 1.
template <typename T, bool CFG, int NT, bool FILT>
__device__ int draw_token(const FinishArgs& a, const Row<T, CFG>& rt, const Row<T, CFG>& rd, PairCtx& ctx, const float u,
                          const int tid, unsigned char* ring, const int ring_bytes, double* tile_sums, FinishSmem& sm,
                          FinishStage& st, uint32_t& phase, int& status, double& Z_out) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int ES = (int)sizeof(T);
  const int lane = tid & 31, warp = tid >> 5;
  const int V = a.V;
  const int ntiles = (V + TILE - 1) / TILE;
  int token = -1;
  Z_out = 0.0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    // ---- Eq. opt_G weights: one fp64 sum per tile ----------------------------------------
    const int n_arr = (ctx.mode == 0 ? 2 : 1) * ARR;
    const int seg_elems = (ring_bytes / n_arr / (TILE * ES)) * TILE;   // elements of each array per segment
    const int slot_bytes = seg_elems * ES;
    for (int x0 = 0; x0 < V; x0 += seg_elems) {
      __syncthreads();   // everybody is done with what the ring held
      const int n = min(seg_elems, V - x0);
      if (tid == 0) {
        fence_before_bulk();
        const uint32_t bytes = (uint32_t)(n * ES);
        mbar_expect_tx(&st.bar, bytes * n_arr);
        bulk_load_row(ring, rt.cond, x0, bytes, V, &st.bar);
        if (CFG) bulk_load_row(ring + slot_bytes, rt.uncond, x0, bytes, V, &st.bar);
        if (ctx.mode == 0) {
          bulk_load_row(ring + ARR * slot_bytes, rd.cond, x0, bytes, V, &st.bar);
          if (CFG) bulk_load_row(ring + (ARR + 1) * slot_bytes, rd.uncond, x0, bytes, V, &st.bar);
        }
      }
      if (!mbar_wait(&st.bar, phase)) status |= 8;
      phase ^= 1u;
      const int seg_tiles = (n + TILE - 1) / TILE;
      // two tiles per warp and trip, so that their reductions overlap
      for (int t0 = warp; t0 < seg_tiles; t0 += 2 * (NT / 32)) {
        float acc2[2] = {0.0f, 0.0f};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int xo = (t0 + r * (NT / 32)) * TILE + lane * VEC;   // offset inside the segment
          if (xo < n) {
            float zt[VEC], zd[VEC];
            unpack_vec<T>(ring + xo * ES, zt);
            if (CFG) {
              float zu[VEC];
              unpack_vec<T>(ring + slot_bytes + xo * ES, zu);
              cfg_mix_vec<VEC>(zt, zu, a.cfg_scale);
            }
            if (ctx.mode == 0) {
              unpack_vec<T>(ring + ARR * slot_bytes + xo * ES, zd);
              if (CFG) {
                float zu[VEC];
                unpack_vec<T>(ring + (ARR + 1) * slot_bytes + xo * ES, zu);
                cfg_mix_vec<VEC>(zd, zu, a.cfg_scale);
              }
            }
            float acc = 0.0f;   // (summed in the order of the scalar form)
#pragma unroll
            for (int k = 0; k < VEC; k += 2) {
              float g0, g1;
              weight_of_pair(FILT ? rt.filter(zt[k]) : zt[k], FILT ? rt.filter(zt[k + 1]) : zt[k + 1],
                             ctx.mode == 0 ? (FILT ? rd.filter(zd[k]) : zd[k]) : 0.0f,
                             ctx.mode == 0 ? (FILT ? rd.filter(zd[k + 1]) : zd[k + 1]) : 0.0f, ctx, g0, g1);
              acc += g0;
              acc += g1;
            }
            acc2[r] = acc;
          }
        }
        double d0 = (double)acc2[0], d1 = (double)acc2[1];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          d0 += __shfl_xor_sync(0xffffffffu, d0, off);
          d1 += __shfl_xor_sync(0xffffffffu, d1, off);
        }
        if (lane == 0) {
          tile_sums[x0 / TILE + t0] = d0;
          if (t0 + NT / 32 < seg_tiles) tile_sums[x0 / TILE + t0 + NT / 32] = d1;
        }
      }
    }
    __syncthreads();
    // ---- locate the tile that holds the crossing C(x) > u Z ---------------------------------
    if (warp == 0) locate_crossing_tile(tile_sums, ntiles, u, lane, sm);
    __syncthreads();
    const double Z = sm.Z;
    if (!(Z > 0.0) || !(Z < (double)CSD_POS_INF)) {
      if (attempt == 0 && ctx.mode == 0) {  // empty positive part: fall back to G := P_j
        ctx.mode = 1;
        status |= 4;
        continue;
      }
      break;  // nothing to draw from
    }
    Z_out = Z;
    // ---- scan inside that tile (its 32 vectors come from global memory again) ------------------
    if (warp == 0) {
      const int tile = sm.pick_tile;
      int tok = -1;
      if (tile >= 0) {   // (the same decision in every lane)
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC], zd[VEC], g[VEC];
        rt.load_tile(x0, V, 1, zt);
        if (ctx.mode == 0) rd.load_tile(x0, V, 1, zd);
#pragma unroll
        for (int k = 0; k < VEC; ++k)
          g[k] = weight_of(FILT ? rt.filter(zt[k]) : zt[k], ctx.mode == 0 ? (FILT ? rd.filter(zd[k]) : zd[k]) : 0.0f, ctx);
        tok = pick_in_tile<VEC>(g, x0, sm.pick_prefix, (double)u * Z, lane);
      }
      if (lane == 0) sm.token = tok;
    }
    __syncthreads();
    token = sm.token;
    break;
  }
  return token;
}

// Writes the distribution a token was drawn from (diagnostic output), or zeros.
template <typename T, bool CFG, int NT>
__device__ void write_G(const FinishArgs& a, const int b, const int j, const SeqRecord& rec, const int tid) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  const int lane = tid & 31, warp = tid >> 5;
  const int V = a.V;
  float* G_out = a.dbg_G + (int64_t)b * V;
  if (rec.token < 0 || !(rec.Z > 0.0)) {
    for (int x = tid; x < V; x += NT) G_out[x] = 0.0f;
    return;
  }
  PairCtx ctx;
  ctx.Mt = rec.Mt; ctx.St = rec.St; ctx.Md = rec.Md; ctx.Sd = rec.Sd;
  ctx.inv_t = 1.0f / (1.0f + ctx.St);
  ctx.inv_den = ctx.inv_t / (1.0f + ctx.Sd);
  ctx.one_minus_omega = rec.one_minus_omega;
  ctx.mode = rec.mode;
  Row<T, CFG> rt = row_at<T, CFG>(a, b, 0, j);
  rt.thr = rec.thr_t;
  Row<T, CFG> rd = rt;
  if (j < a.gamma) { rd = row_at<T, CFG>(a, b, 1, j); rd.thr = rec.thr_d; }
  const float invZ = (float)(1.0 / rec.Z);
  const int ntiles = (V + TILE - 1) / TILE;
  for (int tile = warp; tile < ntiles; tile += NT / 32) {
    const int x0 = tile * TILE + lane * VEC;
    float zt[VEC], zd[VEC];
    rt.load_tile(x0, V, 1, zt);
    if (ctx.mode == 0) rd.load_tile(x0, V, 1, zd);
#pragma unroll
    for (int k = 0; k < VEC; ++k)
      if (x0 + k < V)
        G_out[x0 + k] = weight_of(rt.filter(zt[k]), ctx.mode == 0 ? rd.filter(zd[k]) : 0.0f, ctx) * invZ;
  }
}

// The per-position sums of Theorem 2 (inner sum of Eq. token_exp, bracket of Eq. bd2) for the block's
// positions of sequence b: a second pass over both rows of each position, brought through the two
// halves of the ring by bulk copies (the copies of the next segment run while this one is summed).
// Follows accept_positions of the same sequence (row statistics in sm); reads only the call's inputs
// and leaves the results in st.mon_am / st.mon_bt, so it runs before the block's griddepcontrol.wait.
// red needs two doubles per warp; phase and phase2 are the parities of st.bar and st.bar2.
template <typename T, bool CFG, int NT, bool FILT>
__device__ void position_terms(const FinishArgs& a, const BlockShare& sh, const int b, const int tid,
                               unsigned char* ring, const int ring_bytes, double* red, FinishSmem& sm,
                               FinishStage& st, uint32_t& phase, uint32_t& phase2) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int ES = (int)sizeof(T);
  const int lane = tid & 31, warp = tid >> 5;
  const int V = a.V;
  const int n_arr = 2 * ARR;
  const int buf_bytes = ring_bytes / 2;
  const int seg_elems = (buf_bytes / n_arr / (TILE * ES)) * TILE;   // elements of each array per segment
  const int slot_bytes = seg_elems * ES;
  const int nseg = (V + seg_elems - 1) / seg_elems;
  const int npos = sh.pos_end - sh.pos_begin;
  const int njobs = npos * nseg;   // job j: segment j % nseg of position pos_begin + j / nseg
  auto issue = [&](int j) {        // thread 0; the buffer's last reader is behind a barrier
    const int i = sh.pos_begin + j / nseg;
    if (!(sm.valid[0][i] && sm.valid[1][i])) return;   // nothing is read for an unusable position
    const int x0 = (j % nseg) * seg_elems;
    const uint32_t bytes = (uint32_t)(min(seg_elems, V - x0) * ES);
    unsigned char* buf = ring + (j & 1) * buf_bytes;
    uint64_t* bar = (j & 1) ? &st.bar2 : &st.bar;
    const Row<T, CFG> rt = row_at<T, CFG>(a, b, 0, i), rd = row_at<T, CFG>(a, b, 1, i);
    fence_before_bulk();
    mbar_expect_tx(bar, bytes * n_arr);
    bulk_load_row(buf, rt.cond, x0, bytes, V, bar);
    if (CFG) bulk_load_row(buf + slot_bytes, rt.uncond, x0, bytes, V, bar);
    bulk_load_row(buf + ARR * slot_bytes, rd.cond, x0, bytes, V, bar);
    if (CFG) bulk_load_row(buf + (ARR + 1) * slot_bytes, rd.uncond, x0, bytes, V, bar);
  };
  __syncthreads();   // everybody is done with what the ring held
  if (tid == 0 && njobs > 0) issue(0);
  float am = 0.0f, bt2 = 0.0f;
  for (int j = 0; j < njobs; ++j) {
    const int i = sh.pos_begin + j / nseg;
    const int sg = j % nseg;
    const bool usable = sm.valid[0][i] && sm.valid[1][i];   // (the same decision in every thread)
    if (j > 0) __syncthreads();   // job j-1 has been summed: its buffer takes job j+1
    if (tid == 0 && j + 1 < njobs) issue(j + 1);
    if (usable) {
      if (j & 1) { (void)mbar_wait(&st.bar2, phase2); phase2 ^= 1u; }
      else { (void)mbar_wait(&st.bar, phase); phase ^= 1u; }
      // (a wait that gives up leaves garbage in a diagnostic only)
      TermsCtx tc;
      tc.Mt = sm.M[0][i]; tc.Md = sm.M[1][i];
      tc.inv_t = 1.0f / (1.0f + sm.S[0][i]); tc.inv_d = 1.0f / (1.0f + sm.S[1][i]);
      tc.omega = st.omega[i];
      Row<T, CFG> rt, rd;   // only the thresholds are used here
      rt.thr = sm.thr[0][i];
      rd.thr = sm.thr[1][i];
      const unsigned char* buf = ring + (j & 1) * buf_bytes;
      const int n = min(seg_elems, V - sg * seg_elems);
      for (int xo = tid * VEC; xo < n; xo += NT * VEC) {
        float zt[VEC], zd[VEC];
        unpack_vec<T>(buf + xo * ES, zt);
        unpack_vec<T>(buf + ARR * slot_bytes + xo * ES, zd);
        if (CFG) {
          float zu[VEC];
          unpack_vec<T>(buf + slot_bytes + xo * ES, zu);
          cfg_mix_vec<VEC>(zt, zu, a.cfg_scale);
          unpack_vec<T>(buf + (ARR + 1) * slot_bytes + xo * ES, zu);
          cfg_mix_vec<VEC>(zd, zu, a.cfg_scale);
        }
#pragma unroll
        for (int k = 0; k < VEC; ++k)
          terms_of(FILT ? rt.filter(zt[k]) : zt[k], FILT ? rd.filter(zd[k]) : zd[k], tc, am, bt2);
      }
    }
    if (sg == nseg - 1) {   // the position is complete
      const double wa = warp_sum_double((double)am), wb = warp_sum_double((double)bt2);
      if (lane == 0) { red[2 * warp] = wa; red[2 * warp + 1] = wb; }
      __syncthreads();
      if (tid == 0) {
        double ta = 0.0, tb = 0.0;
        for (int w = 0; w < NT / 32; ++w) { ta += red[2 * w]; tb += red[2 * w + 1]; }
        const float nanv = __int_as_float(0x7fc00000);
        st.mon_am[i] = usable ? (float)ta : nanv;
        st.mon_bt[i] = usable ? (float)(2.0 * tb) : nanv;
      }
      am = 0.0f;
      bt2 = 0.0f;
    }
  }
  __syncthreads();
}

// Tokens, multipliers and uniforms of the block's positions of its sl-th sequence, into shared memory.
// Called for the first sequence when the kernel starts, so that these loads are long complete when
// the accept tests need them.
__device__ __forceinline__ void stage_inputs(const FusedArgs& ua, const BlockShare& sh, const int sl, const int tid,
                                             FinishStage& st) {
  const FinishArgs& a = ua.fin;
  const int L = a.gamma;
  const int b = sh.seq_begin + sl;
  if (b >= sh.seq_end) return;
  if (tid >= sh.pos_begin && tid < sh.pos_end) {
    st.tok[tid] = a.tokens[(int64_t)b * L + tid];
    const float om = a.schedule[tid];
    st.omega[tid] = om >= 0.0f ? om : 0.0f;
    st.uni[tid] = a.uniforms[(int64_t)b * (L + 1) + tid];
  }
  if (tid == L) st.uni[L] = a.uniforms[(int64_t)b * (L + 1) + L];
}

// The block's positions [pos_begin, pos_end) of sequence b: accept tests (Eq. relax) and its first
// rejection (the return value; pos_end if it accepted all of them).  Row statistics come from shared
// memory (rs, local rows of sequence slot sl).  Leaves p, q, f of its positions in st; reads only the
// call's inputs.
template <typename T, bool CFG, int NT>
__device__ int accept_positions(const FusedArgs& ua, const BlockShare& sh, const int sl, const RowStats& rs,
                                const int tid, FinishSmem& sm, FinishStage& st) {
  const FinishArgs& a = ua.fin;
  const int L = a.gamma, V = a.V;
  const int p0 = sh.pos_begin, p1 = sh.pos_end;
  // ---- 0. inputs of these positions and the row statistics, into shared memory -------------------
  if (sl > 0) stage_inputs(ua, sh, sl, tid, st);   // those of the block's first sequence are staged at kernel start
  if (tid < sh.rows_per_seq) {
    int bb, which, i;
    local_row(sh, sl * sh.rows_per_seq + tid, L, bb, which, i);
    const int r_loc = sl * sh.rows_per_seq + tid;
    sm.M[which][i] = rs.ms[r_loc].x;
    sm.S[which][i] = rs.ms[r_loc].y;
    sm.thr[which][i] = a.use_topk ? rs.thr[r_loc] : CSD_NEG_INF;
    st.tokz[which][i] = rs.tokz[r_loc];
  }
  __syncthreads();
  // ---- 1. Eq. relax and the accept test of every owned position ----------------------------------
  if (tid >= p0 && tid < p1) {
    const int i = tid;
    const float M0 = sm.M[0][i], S0 = sm.S[0][i], M1 = sm.M[1][i], S1 = sm.S[1][i];
    const float thr0 = sm.thr[0][i], thr1 = sm.thr[1][i];
    const bool t_ok = M0 > CSD_NEG_INF && M0 < CSD_POS_INF && S0 >= 0.0f && S0 < CSD_POS_INF;
    const bool d_ok = M1 > CSD_NEG_INF && M1 < CSD_POS_INF && S1 >= 0.0f && S1 < CSD_POS_INF;
    sm.valid[0][i] = t_ok; sm.valid[1][i] = d_ok;
    const int tok = st.tok[i];
    const bool tok_ok = tok >= 0 && tok < V;
    int flag = 0;
    float f = 0.0f, p = __int_as_float(0x7fc00000), q = p;
    if (!t_ok || !d_ok) flag = 1;
    else if (!tok_ok) flag = 2;
    else {
      const float zt = st.tokz[0][i], zd = st.tokz[1][i];
      const float dt = (zt < thr0 ? CSD_NEG_INF : zt) - M0;
      const float dd = (zd < thr1 ? CSD_NEG_INF : zd) - M1;
      p = ex2f(dt * kLog2e) / (1.0f + S0);
      q = ex2f(dd * kLog2e) / (1.0f + S1);
      if (dd == CSD_NEG_INF) f = 1.0f;         // q = 0: p/q = +inf, and 0/0 := 1
      else if (dt == CSD_NEG_INF) f = 0.0f;    // p = 0 < q
      else f = fminf(1.0f, st.omega[i] * ex2f((dt - dd) * kLog2e) * ((1.0f + S1) / (1.0f + S0)));
    }
    sm.acc[i] = (st.uni[i] <= f) ? 1 : 0;
    sm.flag[i] = flag;
    st.p[i] = p; st.q[i] = q; st.f[i] = f;
  }
  if (tid == L && sh.bonus) {
    const float M0 = sm.M[0][L], S0 = sm.S[0][L];
    sm.valid[0][L] = M0 > CSD_NEG_INF && M0 < CSD_POS_INF && S0 >= 0.0f && S0 < CSD_POS_INF;
  }
  __syncthreads();
  // ---- 2. this block's first rejection (the for/break of Algorithm 1, on its positions) ----------
  int j = p0;
  while (j < p1 && sm.acc[j]) ++j;
  return j;
}

// The draw at the block's first rejection j (Eq. opt_G) -- or, with j == pos_end in the block that
// owns the bonus row, the bonus draw.  Follows accept_positions of the same sequence; leaves the
// record in st.rec.
template <typename T, bool CFG, int NT, bool FILT>
__device__ void draw_position(const FusedArgs& ua, const BlockShare& sh, const int sl, int j, const int tid,
                              unsigned char* ring, const int ring_bytes, double* tile_sums, FinishSmem& sm,
                              FinishStage& st, uint32_t& phase, const int extra_status) {
  const FinishArgs& a = ua.fin;
  const int L = a.gamma;
  const int b = sh.seq_begin + sl;
  const bool rejected = j < sh.pos_end;
  int status = extra_status & ~8;
  PairCtx ctx;
  bool draw = false;
  if (rejected) {
    status |= sm.flag[j];
    draw = sm.valid[0][j] != 0;
    ctx.mode = sm.valid[1][j] ? 0 : 1;
  } else if (sh.bonus) {
    j = L;
    ctx.mode = 1;
    draw = sm.valid[0][L] != 0;
    if (!draw) status |= 1;
  }
  int token = -1;
  double Z = 0.0;
  Row<T, CFG> rt = row_at<T, CFG>(a, b, 0, min(j, a.T - 1));
  Row<T, CFG> rd = rt;
  if (draw) {
    ctx.Mt = sm.M[0][j]; ctx.St = sm.S[0][j];
    ctx.Md = j < L ? sm.M[1][j] : 0.0f; ctx.Sd = j < L ? sm.S[1][j] : 0.0f;
    ctx.inv_t = 1.0f / (1.0f + ctx.St);
    ctx.inv_den = ctx.inv_t / (1.0f + ctx.Sd);
    ctx.one_minus_omega = 1.0f - (j < L ? st.omega[j] : 0.0f);
    rt.thr = sm.thr[0][j];
    if (j < L) { rd = row_at<T, CFG>(a, b, 1, j); rd.thr = sm.thr[1][j]; }
    else rd = rt;
    token = draw_token<T, CFG, NT, FILT>(a, rt, rd, ctx, st.uni[L], tid, ring, ring_bytes, tile_sums, sm, st, phase,
                                         status, Z);
  }
  if (tid == 0) {
    SeqRecord& rec = st.rec;
    rec.first_rej = rejected ? j : -1;
    rec.token = token;
    rec.status_at = status;
    rec.status_any = extra_status & 8;
    rec.mode = draw ? ctx.mode : 1;
    rec.Mt = draw ? ctx.Mt : 0.0f; rec.St = draw ? ctx.St : 0.0f;
    rec.Md = draw ? ctx.Md : 0.0f; rec.Sd = draw ? ctx.Sd : 0.0f;
    rec.thr_t = rt.thr; rec.thr_d = rd.thr;
    rec.one_minus_omega = draw ? ctx.one_minus_omega : 1.0f;
    rec.Z = Z;
  }
  __syncthreads();
}

// Emits sequence b from the record of the block that decides it (winner): the accepted prefix, the
// drawn token, padding; accepted length; status; optionally the distribution drawn from.
template <typename T, bool CFG, int NT>
__device__ void emit_sequence(const FusedArgs& ua, const int b, const SeqRecord& win, const int status_any,
                              const int tid) {
  const FinishArgs& a = ua.fin;
  const int L = a.gamma;
  const int tau = win.first_rej >= 0 ? win.first_rej : L;
  if (tid <= L) {
    int v = -1;
    if (tid < tau) v = a.tokens[(int64_t)b * L + tid];
    else if (tid == tau) v = win.token;
    a.out_tokens[(int64_t)b * (L + 1) + tid] = v;
  }
  if (tid == 0) {
    if (a.out_accept_len) a.out_accept_len[b] = tau;
    if (a.out_status) a.out_status[b] = win.status_at | status_any;
  }
  if (a.dbg_G) {
    if (tau < a.T) write_G<T, CFG, NT>(a, b, tau, win, tid);
    else for (int x = tid; x < a.V; x += NT) a.dbg_G[(int64_t)b * a.V + x] = 0.0f;
  }
}

// The draw of a sequence whose blocks form a cluster, shared by all of them.  The block that holds the
// first rejection (or, with none, the bonus row) knows what the weights need -- the two rows'
// statistics and thresholds, the multiplier -- and stores that into every block of the cluster; after
// a cluster barrier each block sums Eq. opt_G over its share of the tiles of the two rows (read from
// global memory: L2 hits) and stores the tile sums into the drawing block's shared memory; after a
// second barrier that block locates the crossing, picks the token and leaves the record in st.rec.
// Every block of the cluster calls this, with the same `owner`; a draw that turns out to have an empty
// positive part is redone by the drawing block alone (draw_token).  What a block's own positions
// contributed to the status is passed in `extra_status`.
template <typename T, bool CFG, int NT, bool FILT>
__device__ void cluster_draw(const FusedArgs& ua, const BlockShare& sh, int j, const int owner, const int tid,
                             unsigned char* ring, const int ring_bytes, double* tile_sums, FinishSmem& sm,
                             FinishStage& st, uint32_t& phase, const int extra_status) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  const FinishArgs& a = ua.fin;
  const int L = a.gamma, V = a.V, c = ua.ctas_per_seq;
  const int b = sh.seq_begin;
  const int lane = tid & 31, warp = tid >> 5;
  const bool mine = owner == sh.slot;
  // ---- what is drawn from: published by the drawing block before the exchange's barrier -----------------
  int status = extra_status & ~8;
  bool rejected = false;
  if (mine) {
    rejected = j < sh.pos_end;
    if (rejected) status |= sm.flag[j];
    else if (sh.bonus && !sm.valid[0][L]) status |= 1;
  }
  const uint32_t* share = st.share[owner];
  // ---- every block: its share of the tile sums -----------------------------------------------------
  const int draw = (int)share[0];
  const int jj = (int)share[2];
  PairCtx ctx;
  ctx.mode = (int)share[1];
  ctx.Mt = __uint_as_float(share[3]); ctx.St = __uint_as_float(share[4]);
  ctx.Md = __uint_as_float(share[5]); ctx.Sd = __uint_as_float(share[6]);
  ctx.inv_t = 1.0f / (1.0f + ctx.St);
  ctx.inv_den = ctx.inv_t / (1.0f + ctx.Sd);
  ctx.one_minus_omega = __uint_as_float(share[9]);
  Row<T, CFG> rt = row_at<T, CFG>(a, b, 0, min(jj, a.T - 1));
  Row<T, CFG> rd = rt;
  rt.thr = __uint_as_float(share[7]);
  if (jj < L) { rd = row_at<T, CFG>(a, b, 1, jj); rd.thr = __uint_as_float(share[8]); }
  const int ntiles = (V + TILE - 1) / TILE;
  if (draw) {
    const int t_begin = (int)((long long)ntiles * sh.slot / c), t_end = (int)((long long)ntiles * (sh.slot + 1) / c);
    // (tiles per warp and trip: two, with all loads issued before the first use, measured no faster here and
    // cost the streaming loops registers)
    constexpr int UNR = 1;
    for (int tile0 = t_begin + warp; tile0 < t_end; tile0 += UNR * (NT / 32)) {
      float zt[UNR][VEC], zd[UNR][VEC];
#pragma unroll
      for (int r = 0; r < UNR; ++r) {
        const int tile = tile0 + r * (NT / 32);
        if (tile < t_end) {
          const int x0 = tile * TILE + lane * VEC;
          rt.load_tile(x0, V, 1, zt[r]);
          if (ctx.mode == 0) rd.load_tile(x0, V, 1, zd[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < UNR; ++r) {
        const int tile = tile0 + r * (NT / 32);
        if (tile < t_end) {
          float acc = 0.0f;
#pragma unroll
          for (int e = 0; e < VEC; e += 2) {
            float g0, g1;
            weight_of_pair(FILT ? rt.filter(zt[r][e]) : zt[r][e], FILT ? rt.filter(zt[r][e + 1]) : zt[r][e + 1],
                           ctx.mode == 0 ? (FILT ? rd.filter(zd[r][e]) : zd[r][e]) : 0.0f,
                           ctx.mode == 0 ? (FILT ? rd.filter(zd[r][e + 1]) : zd[r][e + 1]) : 0.0f, ctx, g0, g1);
            acc += g0;
            acc += g1;
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
          if (lane == 0) cluster_store_f64(&tile_sums[tile], (uint32_t)owner, (double)acc);
        }
      }
    }
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (!mine) return;
  // ---- the drawing block: locate, pick, record --------------------------------------------------------
  int token = -1;
  double Z = 0.0;
  if (draw) {
    const float u = st.uni[L];
    if (warp == 0) locate_crossing_tile(tile_sums, ntiles, u, lane, sm);
    __syncthreads();
    Z = sm.Z;
    if (!(Z > 0.0) || !(Z < (double)CSD_POS_INF)) {
      // an empty positive part (or weights that overflowed): the draw is redone from scratch, alone
      token = draw_token<T, CFG, NT, FILT>(a, rt, rd, ctx, u, tid, ring, ring_bytes, tile_sums, sm, st, phase, status, Z);
    } else {
      if (warp == 0) {
        const int tile = sm.pick_tile;
        int tok = -1;
        if (tile >= 0) {
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC], g[VEC];
          rt.load_tile(x0, V, 1, zt);
          if (ctx.mode == 0) rd.load_tile(x0, V, 1, zd);
#pragma unroll
          for (int e = 0; e < VEC; ++e)
            g[e] = weight_of(FILT ? rt.filter(zt[e]) : zt[e], ctx.mode == 0 ? (FILT ? rd.filter(zd[e]) : zd[e]) : 0.0f, ctx);
          tok = pick_in_tile<VEC>(g, x0, sm.pick_prefix, (double)u * Z, lane);
        }
        if (lane == 0) sm.token = tok;
      }
      __syncthreads();
      token = sm.token;
    }
  }
  if (tid == 0) {
    SeqRecord& rec = st.rec;
    rec.first_rej = rejected ? jj : -1;
    rec.token = token;
    rec.status_at = status;
    rec.status_any = extra_status & 8;
    rec.mode = draw ? ctx.mode : 1;
    rec.Mt = draw ? ctx.Mt : 0.0f; rec.St = draw ? ctx.St : 0.0f;
    rec.Md = draw ? ctx.Md : 0.0f; rec.Sd = draw ? ctx.Sd : 0.0f;
    rec.thr_t = rt.thr; rec.thr_d = rd.thr;
    rec.one_minus_omega = draw ? ctx.one_minus_omega : 1.0f;
    rec.Z = Z;
  }
  __syncthreads();
}

// Phase 2 of both kernels.  Entered by the whole block when its row statistics are complete in
// shared memory.  Everything up to the griddepcontrol.wait reads only the call's inputs, so it runs
// beside the previous call on the stream; after it come the few global writes.
//
// With ctas_per_seq > 1 the blocks of a sequence form one cluster.  Each runs the accept tests of its
// own positions and stores what it found -- its first rejection, if any -- into a word of every
// peer's shared memory; after one cluster barrier every block knows which block holds the sequence's
// first rejection (or that there is none: then the last block, which owns the bonus row).  The draw
// is shared (cluster_draw): that block publishes what the weights need, every block sums its share of
// the tiles into that block's shared memory, and it alone picks the token and emits the sequence.  No
// block reads a peer's shared memory, and none writes to it after the last barrier, so blocks leave
// independently.
template <typename T, bool CFG, int NT, bool FILT>
__device__ void finish_block(const FusedArgs& ua, const BlockShare& sh, const RowStats& rs, const int tid,
                             const bool aborted, unsigned char* ring, const int ring_bytes, double* tile_sums,
                             FinishSmem& sm, FinishStage& st) {
  const FinishArgs& a = ua.fin;
  const int L = a.gamma;
  const int extra = aborted ? 8 : 0;
  uint32_t phase = 0, phase2 = 0;
  const bool want_terms = a.diag_am != nullptr || a.diag_bt != nullptr;
  auto write_pqf = [&](int b) {   // diagnostics and monitors of this block's positions
    if (tid >= sh.pos_begin && tid < sh.pos_end) {
      if (a.dbg_p) a.dbg_p[(int64_t)b * L + tid] = st.p[tid];
      if (a.dbg_q) a.dbg_q[(int64_t)b * L + tid] = st.q[tid];
      if (a.dbg_f) a.dbg_f[(int64_t)b * L + tid] = st.f[tid];
      if (a.diag_am) a.diag_am[(int64_t)b * L + tid] = st.mon_am[tid];
      if (a.diag_bt) a.diag_bt[(int64_t)b * L + tid] = st.mon_bt[tid];
    }
  };
  if (ua.ctas_per_seq == 1) {
    // the block owns whole sequences
    int sticky = 0;
    for (int sl = 0; sl < sh.seq_end - sh.seq_begin; ++sl) {
      const int b = sh.seq_begin + sl;
      const int j = accept_positions<T, CFG, NT>(ua, sh, sl, rs, tid, sm, st);
      draw_position<T, CFG, NT, FILT>(ua, sh, sl, j, tid, ring, ring_bytes, tile_sums, sm, st, phase, extra);
      if (want_terms) position_terms<T, CFG, NT, FILT>(a, sh, b, tid, ring, ring_bytes, tile_sums, sm, st, phase, phase2);
      if (sl == 0) {   // before the block's first global write: outputs of consecutive calls stay in order
        pdl_wait();
        sticky = (ua.error_flag && __ldcg(ua.error_flag)) ? 8 : 0;
      }
      write_pqf(b);
      emit_sequence<T, CFG, NT>(ua, b, st.rec, st.rec.status_any | sticky, tid);
      __syncthreads();
    }
    return;
  }
  const int b = sh.seq_begin;
  const int c = ua.ctas_per_seq;
  const int j = accept_positions<T, CFG, NT>(ua, sh, 0, rs, tid, sm, st);
  // ---- tell every block of the sequence: bit 0 rejected, bit 1 a bounded wait gave up ------------
  cluster_wait();   // second half of the barrier begun at kernel start: every peer is running
  if (tid < c) {
    const uint32_t rank = (uint32_t)tid;
    cluster_store(&st.xch[sh.slot], rank, (j < sh.pos_end ? 1u : 0u) | (aborted ? 2u : 0u));
    // ... and, in the same exchange, what the draw's weights need should this block turn out to decide
    // the sequence: the position drawn at (its first rejection, or the bonus row), the two rows'
    // statistics and filter levels, 1 - omega
    int jd = j, draw = 0, mode = 1;
    if (j < sh.pos_end) {
      draw = sm.valid[0][j] != 0;
      mode = sm.valid[1][j] ? 0 : 1;
    } else if (sh.bonus) {
      jd = L;
      draw = sm.valid[0][L] != 0;
    }
    const int jt = min(jd, a.T - 1);
    uint32_t* mine_at = st.share[sh.slot];
    cluster_store(&mine_at[0], rank, (uint32_t)draw);
    cluster_store(&mine_at[1], rank, (uint32_t)mode);
    cluster_store(&mine_at[2], rank, (uint32_t)jd);
    cluster_store(&mine_at[3], rank, __float_as_uint(sm.M[0][jt]));
    cluster_store(&mine_at[4], rank, __float_as_uint(sm.S[0][jt]));
    cluster_store(&mine_at[5], rank, __float_as_uint(jd < L ? sm.M[1][jd] : 0.0f));
    cluster_store(&mine_at[6], rank, __float_as_uint(jd < L ? sm.S[1][jd] : 0.0f));
    cluster_store(&mine_at[7], rank, __float_as_uint(sm.thr[0][jt]));
    cluster_store(&mine_at[8], rank, __float_as_uint(jd < L ? sm.thr[1][jd] : CSD_NEG_INF));
    cluster_store(&mine_at[9], rank, __float_as_uint(1.0f - (jd < L ? st.omega[jd] : 0.0f)));
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  int owner = c - 1, any = 0;
  for (int k = c - 1; k >= 0; --k) {
    const uint32_t w = st.xch[k];
    if (w & 1u) owner = k;
    if (w & 2u) any = 8;
  }
  // the draw is shared by all blocks of the cluster
  cluster_draw<T, CFG, NT, FILT>(ua, sh, j, owner, tid, ring, ring_bytes, tile_sums, sm, st, phase, extra);
  if (owner != sh.slot) {   // another block decides the sequence
    if (a.dbg_p || a.dbg_q || a.dbg_f || want_terms) {
      if (want_terms) position_terms<T, CFG, NT, FILT>(a, sh, b, tid, ring, ring_bytes, tile_sums, sm, st, phase, phase2);
      pdl_wait();
      write_pqf(b);
    }
    return;
  }
  if (want_terms) position_terms<T, CFG, NT, FILT>(a, sh, b, tid, ring, ring_bytes, tile_sums, sm, st, phase, phase2);
  pdl_wait();   // the previous call has completed: outputs of consecutive calls stay in order
  if (ua.error_flag && __ldcg(ua.error_flag)) any = 8;
  write_pqf(b);
  emit_sequence<T, CFG, NT>(ua, b, st.rec, any, tid);
}

// Stats-only calls (FusedArgs::stats_out): the block's rows go to global memory in the row order of the
// multi-launch kernels, after the previous operation on the stream has completed (its finishing kernel
// may still be reading the same arrays).
__device__ __forceinline__ void write_row_stats(const FusedArgs& a, const BlockShare& sh, const RowStats& rs, const int tid,
                                                const int nthreads, const bool aborted) {
  pdl_wait();
  const FinishArgs& f = a.fin;
  for (int r = tid; r < sh.n_rows && r < kBlockRows; r += nthreads) {
    int b, which, i;
    local_row(sh, r, f.gamma, b, which, i);
    const int64_t row_id = (int64_t)b * (f.T + f.gamma) + (which == 0 ? i : f.T + i);
    a.stats_out[row_id] = aborted ? make_float2(__int_as_float(0x7fc00000), 0.0f) : rs.ms[r];   // (a row of a call that
    if (a.thr_out) a.thr_out[row_id] = rs.thr[r];                                              //  gave up reads as unusable)
  }
  if (a.ctas_per_seq > 1) cluster_wait();   // second half of the barrier begun at kernel start
}

// ======================= plain kernel: one pipeline per warp ============================
// A warp owns a contiguous range of items (an item is a part of a row: chunks_per_part warp
// stages), a private ring of kWStages stages of kWStageBytes, issues its own refills, and keeps
// a running (m, s) per lane that it reduces once per item.  Eight such pipelines per block sit
// at different points of their loops and hide each other's latencies; phase 1 has no block-wide
// step at all.
constexpr int kWStages = 2;
constexpr int kWStageBytes = 3072;
constexpr int kBlockStash = 1536;   // items (row parts) a block may own
constexpr int kPlainRingBytes = kPlainWarps * kWStages * kWStageBytes;

struct PlainSmem {
  alignas(128) unsigned char ring[kPlainWarps][kWStages][kWStageBytes];
  alignas(8) uint64_t full[kPlainWarps][kWStages];
  alignas(8) float2 stash[kBlockStash];   // (m, s) per item, by local item index; after the rows' parts have
                                          // been merged, the draw keeps its tile sums here
  RowStats rs;
  int abort;
  FinishSmem fin;
  FinishStage fst;
};
static_assert(sizeof(float2) * kBlockStash >= sizeof(double) * kFinTiles, "tile sums live in the stash");

template <typename T, bool CFG>
__global__ void __launch_bounds__(kPlainThreads, 3) verify_plain_kernel(const FusedArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int EPS = kWStageBytes / ((int)sizeof(T) * ARR);   // elements of a row per warp stage
  constexpr int VPL = EPS / 32;                                // values per lane per stage
  constexpr int NVS = VPL / VEC;                               // 16-byte vectors per lane per stage
  static_assert(NVS >= 1, "a stage holds at least one vector per lane");
  extern __shared__ __align__(128) unsigned char fused_smem_raw[];
  PlainSmem& sm = *reinterpret_cast<PlainSmem*>(fused_smem_raw);

  // the next call on the stream may start: see the head of this file (a stats-only call is followed by
  // its finishing kernel, whose large blocks would only sit on SMs this kernel needs: it follows at exit)
  if (a.stats_out == nullptr) pdl_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const FinishArgs& f = a.fin;
  const int V = f.V;
  const int part_elems = a.chunks_per_part * EPS;
  const int parts = a.parts_per_row;

  if (tid == 0) { sm.abort = 0; mbar_init(&sm.fst.bar, 1); mbar_init(&sm.fst.bar2, 1); }
  if (lane == 0) {
    for (int s = 0; s < kWStages; ++s) mbar_init(&sm.full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (a.ctas_per_seq > 1) cluster_arrive();   // first half; finish_block waits before it writes to a peer

  // the block's items (parts of its local rows, see block_share), split evenly over its warps
  const BlockShare sh = block_share(a);
  const bool stats_only = a.stats_out != nullptr;
  const int n_block = sh.n_rows * parts;
  const int item_begin = (int)((long long)n_block * warp / kPlainWarps);
  const int item_end = (int)((long long)n_block * (warp + 1) / kPlainWarps);

  // producer cursor (meaningful in lane 0): the next chunk to copy
  int p_item = item_begin, p_x = 0, p_xend = 0, p_s = 0;
  int p_count = 0;   // chunks announced to the barriers so far
  int p_row = item_begin / parts, p_part = item_begin - p_row * parts;   // kept incrementally from here on
  const T *p_cond = nullptr, *p_uncond = nullptr;
  // (test aid, see FusedArgs: the warp that owns the block's first item)
  bool drop_next = a.drop_first_copy != 0 && blockIdx.x == 0 && item_begin == 0 && item_end > 0;
  auto producer_open_row = [&]() {    // pointers of row p_row
    int b, which, i;
    local_row(sh, p_row, f.gamma, b, which, i);
    const Row<T, CFG> row = row_at<T, CFG>(f, b, which, i);
    p_cond = row.cond;
    p_uncond = row.uncond;
  };
  auto producer_open_item = [&]() {   // sets the cursor to the first chunk of part p_part of the open row
    p_x = p_part * part_elems;
    p_xend = min(V, p_x + part_elems);
  };
  auto producer_issue = [&]() {       // copies one chunk into the next stage of the ring, if any is left
    if (p_item >= item_end) return;
    const uint32_t bytes = (uint32_t)(min(EPS, p_xend - p_x) * (int)sizeof(T));
    mbar_expect_tx(&sm.full[warp][p_s], bytes * ARR);
    if (!drop_next) {
      bulk_load_row(&sm.ring[warp][p_s][0], p_cond, p_x, bytes, V, &sm.full[warp][p_s]);
      if (CFG) bulk_load_row(&sm.ring[warp][p_s][kWStageBytes / 2], p_uncond, p_x, bytes, V, &sm.full[warp][p_s]);
    }
    drop_next = false;
    ++p_count;
    p_s = p_s + 1 == kWStages ? 0 : p_s + 1;
    p_x += EPS;
    if (p_x >= p_xend) {
      ++p_item;
      if (++p_part == parts) { p_part = 0; ++p_row; if (p_item < item_end) producer_open_row(); }
      if (p_item < item_end) producer_open_item();
    }
  };
  if (lane == 0 && item_begin < item_end) {
    producer_open_row();
    producer_open_item();
    for (int s = 0; s < kWStages; ++s) producer_issue();
  }
  // (the first copies are under way: the block's small inputs and the drafted tokens' logits -- two dependent
  // trips to memory -- are fetched in their shadow)
  if (!stats_only) {
    stage_inputs(a, sh, 0, tid, sm.fst);
    load_token_logits<T, CFG, kPlainThreads>(f, sh, tid, sm.rs);
  }

  // ================================= phase 1 ===========================================
  int n_my = 0;
  {
    int c_s = 0;          // stage the consumer reads next
    uint32_t c_par = 0;   // its parity
    int waited = 0;       // chunks whose copies this lane has seen complete
    bool ok = true;       // false once a wait has run out: from then on nothing is waited for or issued
    int part = item_begin % parts;   // kept incrementally
    for (int item = item_begin; item < item_end; ++item, ++n_my, ++part) {
      if (part == parts) part = 0;
      const int x_begin = part * part_elems;
      const int x_end = min(V, x_begin + part_elems);
      // Running statistics of the item, relative to a maximum that is the same in every lane of
      // the warp: Mw = largest value met so far by any lane, s = this lane's sum of
      // exp(z - Mw) over its values below Mw, cnt = this lane's number of values equal to Mw.
      // Because the reference is warp-uniform, a group of values below it is summed with no
      // test per value, and the exact treatment of values equal to it is a uniform branch
      // taken only where the maximum sits.
      // The exponent (z - Mw) log2(e) is formed by one fused multiply-add, z * log2(e) - MwL with MwL
      // the ROUNDED product Mw * log2(e); its rounding error dlt = Mw * log2(e) - MwL (exact, again by
      // a fused multiply-add) is a common factor 2^dlt of the sum and is divided out once per item.
      float Mw = CSD_NEG_INF, s_run = 0.0f;
      float nMwL = 0.0f, dlt = 0.0f;   // -MwL and dlt of the current reference (while Mw is -inf every value is
                                       // -inf or NaN, and with 0 here its exponential is 0 or NaN as it should be)
      int cnt_run = 0;
      for (int x0 = x_begin; x0 < x_end; x0 += EPS) {
        if (ok) {
          if (mbar_wait(&sm.full[warp][c_s], c_par, a.wait_limit)) ++waited; else ok = false;
        }
        const int n = min(EPS, x_end - x0);
        const unsigned char* stage = &sm.ring[warp][c_s][0];
        const bool full = n == EPS;   // (after a timeout the data is garbage anyway: the call is flagged)
        // The whole stage is one group: its values (packed bf16 pairs where nothing has to be mixed) sit
        // in registers, one reduction gives the warp's largest, and since that result depends on every
        // lane's loads the stage can be handed back for its refill before the exponentials are taken.
        constexpr bool PACKED = !CFG && sizeof(T) == 2;
        constexpr int NW = PACKED ? NVS * 4 : 1;
        constexpr int NF = PACKED ? 1 : NVS * VEC;
        uint32_t w[NW];
        float vals[NF];
        float gm;   // this lane's largest value of the stage
        if (PACKED && full) {
#pragma unroll
          for (int v = 0; v < NVS; ++v) {
            const uint4 q4 = *reinterpret_cast<const uint4*>(stage + (v * 32 + lane) * VEC * (int)sizeof(T));
            w[(v * 4 + 0) % NW] = q4.x; w[(v * 4 + 1) % NW] = q4.y; w[(v * 4 + 2) % NW] = q4.z; w[(v * 4 + 3) % NW] = q4.w;
          }
          uint32_t m2[4] = {w[0], w[1 % NW], w[2 % NW], w[3 % NW]};
#pragma unroll
          for (int k = 4; k < NW; ++k) asm("max.bf16x2 %0, %0, %1;" : "+r"(m2[k & 3]) : "r"(w[k]));
          asm("max.bf16x2 %0, %0, %1;" : "+r"(m2[0]) : "r"(m2[1]));
          asm("max.bf16x2 %0, %0, %1;" : "+r"(m2[2]) : "r"(m2[3]));
          asm("max.bf16x2 %0, %0, %1;" : "+r"(m2[0]) : "r"(m2[2]));
          gm = fmaxf(__uint_as_float(m2[0] << 16), __uint_as_float(m2[0] & 0xffff0000u));
        } else if (PACKED) {
          // ragged last stage of a packed row: out-of-range pairs read as -inf (0xff80 twice)
#pragma unroll
          for (int v = 0; v < NVS; ++v) {
            const int xo = (v * 32 + lane) * VEC;
            uint4 q4 = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
            if (xo < n) q4 = *reinterpret_cast<const uint4*>(stage + xo * (int)sizeof(T));
            w[(v * 4 + 0) % NW] = q4.x; w[(v * 4 + 1) % NW] = q4.y; w[(v * 4 + 2) % NW] = q4.z; w[(v * 4 + 3) % NW] = q4.w;
          }
          uint32_t m2 = w[0];
#pragma unroll
          for (int k = 1; k < NW; ++k) asm("max.bf16x2 %0, %0, %1;" : "+r"(m2) : "r"(w[k]));
          gm = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
        } else {
#pragma unroll
          for (int v = 0; v < NVS; ++v) {
            const int xo = (v * 32 + lane) * VEC;
            float zc[VEC];
            if (full || xo < n) {
              unpack_vec<T>(stage + xo * (int)sizeof(T), zc);
              if (CFG) {
                float zu[VEC];
                unpack_vec<T>(stage + kWStageBytes / 2 + xo * (int)sizeof(T), zu);
                cfg_mix_vec<VEC>(zc, zu, f.cfg_scale);
              }
            } else {
#pragma unroll
              for (int e = 0; e < VEC; ++e) zc[e] = CSD_NEG_INF;
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e) vals[(v * VEC + e) % NF] = zc[e];
          }
          float m4[4] = {CSD_NEG_INF, CSD_NEG_INF, CSD_NEG_INF, CSD_NEG_INF};
#pragma unroll
          for (int e = 0; e < NF; ++e) m4[e & 3] = fmaxf(m4[e & 3], vals[e]);
          gm = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        }
        // the stage's largest value over the warp (one integer reduction on order-preserving keys)
        int key = __float_as_int(gm);
        key ^= (key >> 31) & 0x7fffffff;
        key = __reduce_max_sync(0xffffffffu, key);
        key ^= (key >> 31) & 0x7fffffff;
        const float wm = __int_as_float(key);
        if (lane == 0 && ok) {   // every lane has read the stage: refill it with the chunk kWStages ahead
          fence_before_bulk();
          producer_issue();
        }
        if (wm > Mw) {   // a new maximum: what was counted as "equal to the maximum" becomes ordinary mass
          const float MwL = wm * kLog2e;
          const float dlt_new = fmaf(wm, kLog2e, -MwL);
          s_run = (s_run * ex2f(-dlt) + (float)cnt_run) * ex2f((Mw - wm) * kLog2e) * ex2f(dlt_new);
          cnt_run = 0;
          Mw = wm;
          nMwL = -MwL;
          dlt = dlt_new;
        }
        float acc4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (PACKED) {
          if (wm == Mw) {
            // values equal to the reference may be present: they are counted, not summed.  On the packed
            // pairs: one compare per pair marks them, the marked halves become -inf (their exponential is
            // then exactly 0) and are counted, 16 bits of the counter per half.
            const uint32_t m16 = __float_as_uint(Mw) >> 16;
            const uint32_t Mw2 = m16 | (m16 << 16);
            uint32_t c2 = 0;
#pragma unroll
            for (int k = 0; k < NW; k += 2) {
              uint32_t e0, e1;
              asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(e0) : "r"(w[k]), "r"(Mw2));
              asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(e1) : "r"(w[(k + 1) % NW]), "r"(Mw2));
              w[k] = (w[k] & ~e0) | (0xff80ff80u & e0);
              w[(k + 1) % NW] = (w[(k + 1) % NW] & ~e1) | (0xff80ff80u & e1);
              c2 += (e0 & 0x00010001u) + (e1 & 0x00010001u);
            }
            static_assert(NW % 2 == 0 || NW == 1, "pairs of words");
            cnt_run += (int)((c2 & 0xffffu) + (c2 >> 16));
          }
          // exponents and sums two values per instruction (each half the IEEE operation: the same bits as
          // the scalar form); NaN values poison the sum, which marks the row
          const uint64_t l2e2 = pack2(kLog2e, kLog2e), nm2 = pack2(nMwL, nMwL);
          uint64_t accp[2] = {pack2(0.0f, 0.0f), pack2(0.0f, 0.0f)};
#pragma unroll
          for (int k = 0; k < NW; ++k) {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xffff0000u)), l2e2, nm2), x0, x1);
            accp[k & 1] = add2(accp[k & 1], pack2(ex2f(x0), ex2f(x1)));
          }
          unpack2(accp[0], acc4[0], acc4[1]);
          unpack2(accp[1], acc4[2], acc4[3]);
        } else if (wm == Mw) {
          // (branch-free: the exponential of a value equal to the reference is replaced by 0)
          int c4[4] = {0, 0, 0, 0};
#pragma unroll
          for (int e = 0; e < NF; ++e) {
            const float ex = ex2f(fmaf(vals[e], kLog2e, nMwL));
            acc4[e & 3] += vals[e] == Mw ? 0.0f : ex;
            c4[e & 3] += vals[e] == Mw ? 1 : 0;
          }
          cnt_run += (c4[0] + c4[1]) + (c4[2] + c4[3]);
        } else {
#pragma unroll
          for (int e = 0; e < NF; ++e) acc4[e & 3] += ex2f(fmaf(vals[e], kLog2e, nMwL));
        }
        s_run += (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]);
        if (++c_s == kWStages) { c_s = 0; c_par ^= 1u; }
      }
      // the item's pair: m = Mw, s = sum over everything except one entry at the maximum
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        s_run += __shfl_xor_sync(0xffffffffu, s_run, off);
        cnt_run += __shfl_xor_sync(0xffffffffu, cnt_run, off);
      }
      if (lane == 0 && item < kBlockStash) sm.stash[item] = make_float2(Mw, s_run * ex2f(-dlt) + (float)(cnt_run - 1));
    }
    if (!ok) {
      sm.abort = 1;
      if (lane == 0) {
        if (a.error_flag) atomicExch(a.error_flag, 1);
        // Nothing was issued after lane 0's failed wait, so the copies that may still be in flight are
        // those of chunks [waited, p_count): at most one per stage.  Wait for each, again bounded.
        for (int c = waited; c < p_count; ++c)
          (void)mbar_wait(&sm.full[warp][c % kWStages], (uint32_t)(c / kWStages) & 1u, a.wait_limit);
      }
    }
  }

  // ================================= phase 2 ===========================================
  __syncthreads();
  // the statistics of each local row: its parts merged by one warp
  for (int r = warp; r < sh.n_rows; r += kPlainWarps) {
    float m = CSD_NEG_INF, s_acc = -1.0f;
    for (int pp = lane; pp < parts; pp += 32) {
      const float2 v = sm.stash[r * parts + pp];
      stat_merge(m, s_acc, v.x, v.y);
    }
    stat_warp_allreduce(m, s_acc);
    if (lane == 0) { sm.rs.ms[r] = make_float2(m, s_acc); sm.rs.thr[r] = CSD_NEG_INF; }
  }
  __syncthreads();
  if (stats_only) {
    write_row_stats(a, sh, sm.rs, tid, kPlainThreads, sm.abort != 0);
    return;
  }
  finish_block<T, CFG, kPlainThreads, false>(a, sh, sm.rs, tid, sm.abort != 0, &sm.ring[0][0][0], kPlainRingBytes,
                                      reinterpret_cast<double*>(&sm.stash[0]), sm.fin, sm.fst);
}

// ======================= top-k kernel: a block streams whole rows ========================
constexpr int kTkStages = 2;
constexpr int kTkStageBytes = 16384;
constexpr int kTkRingBytes = kTkStages * kTkStageBytes;
constexpr int kWarpList = 256;                // per-warp capacity of the list of values >= lo: the instance that
                                              // leaves room for four blocks per SM ...
constexpr int kWarpListLarge = 512;           // ... and the one for larger k (four as well, with 300 bytes to spare)
constexpr int kLinBins = 512;
constexpr int kCandCap = 64;
constexpr float kLinRangeSigmas = 4.75f;      // the histogram spans [lo, lo + this many deviations)

// bin of v >= lo in the linear histogram; the same instructions wherever it is evaluated
__device__ __forceinline__ int lin_bin(float v, float lo, float scale) {
  return min(kLinBins - 1, (int)__fmul_rn(__fsub_rn(v, lo), scale));
}

template <int WL>
struct TopkSmemT {
  alignas(128) unsigned char ring[kTkStages][kTkStageBytes];
  alignas(8) uint64_t full[kTkStages];
  int readers_done[kTkStages];      // warps that have finished reading the stage's current contents
  int issued_q;                     // chunks announced to the barriers so far (written by the issuing thread)
  alignas(16) int hist[kLinBins];   // linear histogram; first 256 bins double as the radix histogram
  alignas(8) float list[kTopkWarps][WL];   // per warp: the values >= lo it met (the finish keeps its tile sums here)
  int wpos[kTopkWarps];            // per warp: next free slot of its list (may run past the capacity)
  float cand[kCandCap];             // values in the bin of the k-th largest
  int n_cand[2];                    // by row parity
  alignas(16) float mom[2][kTopkWarps];   // per warp: sum and sum of squares of its sampled values
  float wmax[kTopkWarps];
  // per warp, by row parity: sum of exp(z - max) over kept non-maximum values and number of kept values
  // equal to the maximum; the extra slot takes the values of the bin that holds the threshold
  float part_acc[2][kTopkWarps];
  int part_cmax[2][kTopkWarps];
  // the short cut (see the kernel): per warp (m, s) of its whole list, its count of values above the
  // upper level and of values above the drafted token's logit
  float fw_m[kTopkWarps], fw_s[kTopkWarps];
  int fw_cgt[kTopkWarps], fw_rk[kTopkWarps];
  int short_on;                     // cleared once a row has failed the short cut's test: the block stops trying
  int row_short;                    // this row was settled by the short cut
  int short_fail;                   // rows that failed the short cut's test so far
  int bc_i[4];
  int arrive[2];                    // warps that have finished the first / the second pass over their lists
  float row_mx;                     // set by the warp that picks the bin: the row maximum, and whether the
  int row_fast;                     //   gathered lists can be used for this row
  unsigned need_exact[(kBlockRows + 31) / 32];   // rows to be selected exactly from global memory, after the loop
  float red_f[kTopkWarps][2];
  RowStats rs;
  int abort;
  FinishSmem fin;
  FinishStage fst;
  float c_kind[2];                  // by row parity (target / drafter rows alternate): the multiplier of the
                                    //   deviation in the guess, adapted from the rows already done
  float row_mean[2], row_dev[2];    // by row parity: the sample's moments (for that adaptation)
  int adapt_on;                     // set once a guess has missed: from then on every row adapts the multiplier
};
using TopkSmem = TopkSmemT<kWarpList>;

// Bin (of kLinBins, counted in `hist`) that holds the k-th largest value, found by one warp:
// 16 bins per lane from the top, a warp scan, then a second scan inside the owner's 16 bins.
// *rank_in_bin gets the 1-based rank of the answer among the bin's values, from the top.
__device__ __forceinline__ int warp_pick_bin(const int* hist, int k, int lane, int* rank_in_bin) {
  constexpr int PER = kLinBins / 32;           // 16
  const int hi = kLinBins - lane * PER;        // lane 0 owns the top bins [hi - PER, hi)
  int local = 0;
  {
    const int4* v = reinterpret_cast<const int4*>(hist + hi - PER);
#pragma unroll
    for (int q4 = 0; q4 < PER / 4; ++q4) {
      const int4 t = v[q4];
      local += t.x + t.y + t.z + t.w;
    }
  }
  int incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  const unsigned ballot = __ballot_sync(0xffffffffu, incl >= k);
  const int owner = ballot ? __ffs(ballot) - 1 : 31;
  const int above_owner = __shfl_sync(0xffffffffu, incl - local, owner);
  const int owner_hi = kLinBins - owner * PER;
  // second level: lane l < PER looks at bin owner_hi - 1 - l
  const int val = lane < PER ? hist[owner_hi - 1 - lane] : 0;
  int incl2 = val;
#pragma unroll
  for (int off = 1; off < PER; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl2, off);
    if (lane >= off) incl2 += t;
  }
  const unsigned b2 = __ballot_sync(0xffffffffu, lane < PER && above_owner + incl2 >= k);
  const int pick = b2 ? __ffs(b2) - 1 : PER - 1;
  const int before = __shfl_sync(0xffffffffu, above_owner + incl2 - val, pick);
  *rank_in_bin = k - before;
  return owner_hi - 1 - pick;
}

// Exact threshold and filtered statistics of one row read again from global memory: radix
// select over order-preserving keys (four 8-bit digits), then one pass for (m, s).  All
// threads of the block take part; the results are valid in thread 0.
template <typename T, bool CFG, typename SM>
__device__ void exact_row_from_global(const Row<T, CFG>& row, int V, int k, SM& sm, int tid, float& out_m,
                                      float& out_s, float& out_thr) {
  constexpr int VEC = Elem<T>::kVec;
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0, mask = 0;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) sm.hist[tid] = 0;
    __syncthreads();
    for (int x0 = tid * VEC; x0 < V; x0 += kTopkThreads * VEC) {
      float z[VEC];
      row.load_vec(x0, z);
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        const uint32_t key = order_key(z[e]);
        if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 255], 1);
      }
    }
    __syncthreads();
    if (warp == 0) {
      int above;
      const int bin = select_bin_from_top(sm.hist, 256, k, lane, &above);
      if (lane == 0) { sm.bc_i[0] = (int)(prefix | ((uint32_t)bin << shift)); sm.bc_i[1] = k - above; }
    }
    __syncthreads();
    prefix = (uint32_t)sm.bc_i[0];
    k = sm.bc_i[1];
    mask |= 255u << shift;
    __syncthreads();
  }
  const float thr = order_value(prefix);
  float m = CSD_NEG_INF, s = -1.0f;
  for (int x0 = tid * VEC; x0 < V; x0 += kTopkThreads * VEC) {
    float z[VEC];
    row.load_vec(x0, z);
#pragma unroll
    for (int e = 0; e < VEC; ++e) z[e] = z[e] < thr ? CSD_NEG_INF : z[e];
    float m1, s1;
    stat_of_values(z, m1, s1);
    stat_merge(m, s, m1, s1);
  }
  stat_warp_allreduce(m, s);
  if (lane == 0) { sm.red_f[warp][0] = m; sm.red_f[warp][1] = s; }
  __syncthreads();
  if (tid == 0) {
    float mm = sm.red_f[0][0], sv = sm.red_f[0][1];
#pragma unroll
    for (int w = 1; w < kTopkWarps; ++w) stat_merge(mm, sv, sm.red_f[w][0], sm.red_f[w][1]);
    out_m = mm; out_s = sv; out_thr = thr;
  }
  __syncthreads();
}

// One stage of a row as this thread sees it: its NVS 16-byte vectors of the (mixed) row, unpacked
// to fp32.  `base` is the shared address of the stage plus 16 bytes per thread; vector v of the
// thread sits 4096 bytes further per v, the unconditional array half a stage further.  n is the
// number of valid elements in the stage (a multiple of the vector width); what lies beyond reads -inf.
template <typename T, bool CFG, int NVS, bool RAGGED>
__device__ __forceinline__ void load_stage(const uint32_t base, const int n, const int tid, const float scale,
                                           float (&z)[NVS * Elem<T>::kVec]) {
  constexpr int VEC = Elem<T>::kVec;
  auto lds128 = [](uint32_t addr, uint32_t (&w)[4]) {
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
  };
  auto unpack = [](const uint32_t (&w)[4], float (&out)[VEC]) {
    if (sizeof(T) == 4) {
#pragma unroll
      for (int k = 0; k < 4; ++k) out[k] = __uint_as_float(w[k]);
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        out[2 * k] = __uint_as_float(w[k] << 16);
        out[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
      }
    }
  };
#pragma unroll
  for (int v = 0; v < NVS; ++v) {
    float zc[VEC];
    if (!RAGGED || (v * kTopkThreads + tid) * VEC < n) {
      uint32_t w[4];
      lds128(base + v * (kTopkThreads * 16), w);
      unpack(w, zc);
      if (CFG) {
        float zu[VEC];
        lds128(base + kTkStageBytes / 2 + v * (kTopkThreads * 16), w);
        unpack(w, zu);
        cfg_mix_vec<VEC>(zc, zu, scale);
      }
    } else {
#pragma unroll
      for (int e = 0; e < VEC; ++e) zc[e] = CSD_NEG_INF;
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) z[v * VEC + e] = zc[e];
  }
}

// RAGGED: V is not a whole number of stages, so the last stage of a row is partly filled (the host
// picks the instance; without it the streaming loop has no bounds tests at all).
template <typename T, bool CFG, bool RAGGED, int WL>
__global__ void __launch_bounds__(kTopkThreads, 4) verify_topk_kernel(const FusedArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int ES = (int)sizeof(T);
  constexpr int EPS = kTkStageBytes / (ES * ARR);               // elements of a row per stage
  constexpr int VPT = EPS / kTopkThreads;                       // values per thread per stage
  constexpr int NVS = VPT / VEC;                                // 16-byte vectors per thread per stage
  static_assert(kTkStages == 2, "stage and parity of a chunk are taken from the low bits of its index");
  extern __shared__ __align__(128) unsigned char fused_smem_raw[];
  using Smem = TopkSmemT<WL>;
  constexpr int kListCap = kTopkWarps * WL;
  Smem& sm = *reinterpret_cast<Smem*>(fused_smem_raw);

  // the next call on the stream may start: see the head of this file (a stats-only call is followed by
  // its finishing kernel, whose large blocks would only sit on SMs this kernel needs: it follows at exit)
  if (a.stats_out == nullptr) pdl_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const FinishArgs& f = a.fin;
  const int V = f.V;
  const int cpr = (V + EPS - 1) / EPS;   // stages per row
  const int k_top = a.top_k;

  if (tid == 0) {
    for (int s = 0; s < kTkStages; ++s) { mbar_init(&sm.full[s], 1); sm.readers_done[s] = 0; }
    mbar_init(&sm.fst.bar, 1); mbar_init(&sm.fst.bar2, 1);
    sm.abort = 0;
    sm.issued_q = 0;
    sm.n_cand[0] = 0;
    sm.n_cand[1] = 0;
    sm.arrive[0] = 0;
    sm.arrive[1] = 0;
    sm.c_kind[0] = a.lo_sigmas;
    sm.c_kind[1] = a.lo_sigmas;
    sm.adapt_on = 0;
    sm.short_on = (a.hi_delta == a.hi_delta && a.fin.dbg_G == nullptr) ? 1 : 0;
    sm.row_short = 0;
    sm.short_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < (kBlockRows + 31) / 32) sm.need_exact[tid] = 0u;
  __syncthreads();
  if (a.ctas_per_seq > 1) cluster_arrive();   // first half; finish_block waits before it writes to a peer

  // this block's local rows (see block_share)
  const BlockShare sh = block_share(a);
  const bool stats_only = a.stats_out != nullptr;
  const int n_rows = sh.n_rows;
  const int n_chunks = n_rows * cpr;

  auto row_of = [&](int row_id) -> Row<T, CFG> {
    int b, which, i;
    local_row(sh, row_id, f.gamma, b, which, i);
    return row_at<T, CFG>(f, b, which, i);
  };
  // Issues the copies of chunk q of this block (chunk q % cpr of its local row q / cpr), if there is
  // one, into stage q % 2.  One thread at a time per stage.
  auto issue_chunk = [&](int q) {
    if (q >= n_chunks) return;
    const int j = q / cpr, c = q - j * cpr;
    const Row<T, CFG> row = row_of(j);
    const int s = q & 1;
    const int x0 = c * EPS;
    const uint32_t bytes = (uint32_t)(min(EPS, V - x0) * ES);
    mbar_expect_tx(&sm.full[s], bytes * ARR);
    atomicMax(&sm.issued_q, q + 1);
    if (q == 0 && a.drop_first_copy != 0 && blockIdx.x == 0) return;   // (test aid, see FusedArgs)
    bulk_load_row(&sm.ring[s][0], row.cond, x0, bytes, V, &sm.full[s]);
    if (CFG) bulk_load_row(&sm.ring[s][kTkStageBytes / 2], row.uncond, x0, bytes, V, &sm.full[s]);
  };
  if (tid == 0) {
    issue_chunk(0);
    issue_chunk(1);
  }
  // (the first copies are under way: the block's small inputs and the drafted tokens' logits -- two dependent
  // trips to memory -- are fetched in their shadow)
  if (!stats_only) {
    stage_inputs(a, sh, 0, tid, sm.fst);
    load_token_logits<T, CFG, kTopkThreads>(f, sh, tid, sm.rs);
  } else {
    for (int r = tid; r < kBlockRows; r += kTopkThreads) sm.rs.tokz[r] = 0.0f;   // (read by the short cut's rank, unused here)
  }

  // ================================= phase 1 ===========================================
  {
    int q = 0;        // chunks consumed so far
    int waited = 0;   // chunks whose copies this thread has seen complete
    bool ok = true;   // false once a wait has run out: from then on this thread waits for nothing
    const uint32_t ring_mine = smem_addr(&sm.ring[0][0]) + (uint32_t)tid * 16u;
    const uint32_t list_mine = smem_addr(&sm.list[warp][0]);
    const uint32_t hist_addr = smem_addr(&sm.hist[0]);
    const uint32_t lanemask_lt = (1u << lane) - 1u;
    for (int r = 0; r < n_rows; ++r) {
      const int par = r & 1;
      float lo = 0.0f, scale = 0.0f, dev = 0.0f;
      uint32_t wcur = 0;   // next free slot of the warp's list (may run past the capacity)
      reinterpret_cast<int2*>(sm.hist)[tid] = make_int2(0, 0);
      static_assert(kLinBins == 2 * kTopkThreads, "every thread clears two bins");
      for (int c = 0; c < cpr; ++c, ++q) {
        const int s = q & 1;
        if (ok) {
          if (mbar_wait(&sm.full[s], (uint32_t)(q >> 1) & 1u, a.wait_limit)) ++waited;
          else { ok = false; *(volatile int*)&sm.abort = 1; }
        }
        const int n = RAGGED ? min(EPS, V - c * EPS) : EPS;
        float z[VPT];
        load_stage<T, CFG, NVS, RAGGED>(ring_mine + (uint32_t)s * kTkStageBytes, n, tid, f.cfg_scale, z);
        __syncwarp();
        if (lane == 0) {   // this warp is done with the stage; the last one to say so refills it
          __threadfence_block();
          if (atom_add_shared(&sm.readers_done[s], 1) == kTopkWarps - 1) {
            sm.readers_done[s] = 0;
            __threadfence_block();
            // (a thread that gave up set the flag before it counted itself here: once any wait has
            // run out, nothing more is issued)
            if (*(volatile int*)&sm.abort == 0) {
              fence_before_bulk();
              issue_chunk(q + kTkStages);
            }
          }
        }
        if (c == 0) {
          // The first stage is the sample for the threshold guess: its mean, and as its scale the mean
          // ABSOLUTE deviation (each warp about its own mean, over every other 16-byte vector of the
          // sample), which heavy-tailed logits do not throw about from row to row the way they do the
          // standard deviation -- and in whose units the upper quantiles of a Gaussian and of a
          // Student-t with three degrees of freedom nearly coincide, so one multiplier serves both.
          float sum1 = 0.0f, sum2 = 0.0f, sum2b = 0.0f;
          uint64_t sum1p = pack2(0.0f, 0.0f);   // (two values per addition)
          int mine_n = 0;
#pragma unroll
          for (int v = 0; v < NVS; ++v) {
            if (!RAGGED || (v * kTopkThreads + tid) * VEC < n) {
#pragma unroll
              for (int e = 0; e < VEC; e += 2) sum1p = add2(sum1p, pack2(z[v * VEC + e], z[v * VEC + e + 1]));
              mine_n += VEC;
            }
          }
          { float s_lo, s_hi; unpack2(sum1p, s_lo, s_hi); sum1 = s_lo + s_hi; }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) sum1 += __shfl_xor_sync(0xffffffffu, sum1, off);
          const float wmean = RAGGED ? sum1 * rcp_approx((float)max(1, __reduce_add_sync(0xffffffffu, mine_n)))
                                     : sum1 * (1.0f / (float)(32 * VPT));
          const uint64_t nwm2 = pack2(-wmean, -wmean);
          int dev_n = 0;   // values this thread put into the deviation sum
#pragma unroll
          for (int v = 0; v < NVS; v += 2) {
            if (!RAGGED || (v * kTopkThreads + tid) * VEC < n) {
#pragma unroll
              for (int e = 0; e < VEC; e += 2) {
                float d0, d1;
                unpack2(add2(pack2(z[v * VEC + e], z[v * VEC + e + 1]), nwm2), d0, d1);
                sum2 += fabsf(d0);
                sum2b += fabsf(d1);
              }
              dev_n += VEC;
            }
          }
          sum2 += sum2b;
          // (the sum goes to the block as a mean over the warp's share, scaled back to the sample's size)
          {
            float cntf = RAGGED ? (float)dev_n : (float)(VEC * ((NVS + 1) / 2));
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
              sum2 += __shfl_xor_sync(0xffffffffu, sum2, off);
              if (RAGGED) cntf += __shfl_xor_sync(0xffffffffu, cntf, off);
            }
            if (!RAGGED) cntf *= 32.0f;
            const float warp_n = RAGGED ? (float)__reduce_add_sync(0xffffffffu, mine_n) : (float)(32 * VPT);
            sum2 = cntf > 0.0f ? sum2 * (warp_n * rcp_approx(cntf)) : 0.0f;
          }
          if (lane == 0) { sm.mom[0][warp] = sum1; sm.mom[1][warp] = sum2; }
          __syncthreads();   // ---- S0: moments, cleared histogram and list cursors; the previous row is complete
          if (tid == 0) sm.n_cand[par ^ 1] = 0;   // for the next row; nobody reads the previous row's count any more
          float s1 = 0.0f, s2 = 0.0f;
          {
            const float4* m4 = reinterpret_cast<const float4*>(&sm.mom[0][0]);
            static_assert(kTopkWarps == 8, "the moments of eight warps are four 16-byte loads");
            const float4 a0 = m4[0], a1 = m4[1], b0 = m4[2], b1 = m4[3];
            s1 = ((a0.x + a0.y) + (a0.z + a0.w)) + ((a1.x + a1.y) + (a1.z + a1.w));
            s2 = ((b0.x + b0.y) + (b0.z + b0.w)) + ((b1.x + b1.y) + (b1.z + b1.w));
          }
          // (a guess: approximate reciprocal and root are enough, every thread gets the same bits)
          const float inv_n = RAGGED ? rcp_approx((float)n) : 1.0f / (float)EPS;
          const float mean = s1 * inv_n;
          // (sqrt(pi / 2) x mean absolute deviation is the standard deviation, were the row Gaussian)
          dev = 1.2533141f * (s2 * inv_n);
          lo = mean + sm.c_kind[par] * dev;
          scale = ((float)kLinBins / kLinRangeSigmas) * rcp_approx(dev);
          if (tid == 0) { sm.row_mean[par] = mean; sm.row_dev[par] = dev; }
        }
        // ---- gather this stage's values >= lo into the warp's list -------------------------
        // (the test is "not below lo", so that a NaN lands in the list and marks the row through the
        // maximum).  One bit per value in a mask, the slots from a prefix over the lanes' counts, then
        // the flagged values are stored.
        // (the bit is the sign of z - lo, taken two values per subtraction and shifted into the mask by a
        // funnel shift: a NaN difference is the canonical, positive NaN, and x - x is +0, so both count
        // as "not below")
        uint32_t below_lo = 0;
        {
          const uint64_t nlo2 = pack2(-lo, -lo);
#pragma unroll
          for (int e = VPT - 2; e >= 0; e -= 2) {
            float d0, d1;
            unpack2(add2(pack2(z[e], z[e + 1]), nlo2), d0, d1);
            below_lo = __funnelshift_l(__float_as_uint(d1), below_lo, 1);
            below_lo = __funnelshift_l(__float_as_uint(d0), below_lo, 1);
          }
        }
        const uint32_t mask = ~below_lo & (VPT == 32 ? 0xffffffffu : ((1u << (VPT & 31)) - 1u));
        // slots: the warp's cursor lives in a register (the list is the warp's own); a lane's offset is
        // the sum of the counts of the lanes below it, taken bit by bit from a few ballots
        const uint32_t cnt = (uint32_t)__popc(mask);
        uint32_t below = 0;
        constexpr int kCntBits = VPT <= 15 ? 4 : (VPT <= 31 ? 5 : 6);
        static_assert(VPT <= 63, "a lane's count fits six bits");
#pragma unroll
        for (int bit = 0; bit < kCntBits; ++bit) {
          const uint32_t bal = __ballot_sync(0xffffffffu, (cnt >> bit) & 1u);
          below += (uint32_t)__popc(bal & lanemask_lt) << bit;
        }
        const uint32_t total = __reduce_add_sync(0xffffffffu, cnt);
        const uint32_t pos = wcur + below;
        wcur += total;
        if (pos + cnt <= (uint32_t)WL) {
          uint32_t addr = list_mine + 4u * pos;
#pragma unroll
          for (int e = 0; e < VPT; ++e) {
            if (mask & (1u << e)) {
              asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(z[e]) : "memory");
              addr += 4u;
            }
          }
        }
      }
      // ---- first pass over this warp's list: maximum and histogram -----------------------------
      // (the row maximum is among the gathered values whenever the lists can be used).  The list is
      // padded with -inf to a whole number of 32 slots, so that the passes run without bounds tests.
      if (lane == 0) sm.wpos[warp] = (int)wcur;   // (the warps that settle the row read every warp's count)
      __syncwarp();
      const int wc = (int)wcur;
      int wcp = 0;   // padded length; 0 if the list overflowed (the row is then selected exactly)
      if (wc <= WL) {
        wcp = (wc + 31) & ~31;
        if (wc + lane < wcp) sm.list[warp][wc + lane] = CSD_NEG_INF;
      }
      __syncwarp();
      // ---- the short cut: no threshold at all --------------------------------------------------
      // If a level `hi` a little above lo has fewer than k values above it, the k-th largest value lies
      // in [lo, hi], and the values the filter drops among those gathered all lie there too.  Where
      // their total weight -- at most (gathered - k) * exp(hi - max) -- is below 2^-26 of the row's
      // normaliser, dropping them or not changes nothing that fp32 can see: the row's (m, s) is that
      // of ALL gathered values, lo itself serves as the threshold from here on (for the draw's filter
      // and the diagnostics: what it lets through beyond the exact filter has weight below 1e-7 of an
      // ulp), and whether the drafted token survives the exact filter is decided by its exact rank
      // (fewer than k gathered values above its logit).  One pass over the lists and one barrier
      // instead of a histogram, a selection and two barriers; rows that fail the test (flat rows,
      // where the values near the threshold carry weight) take the full selection below, on the same
      // lists; after three such rows the block stops trying.
      if (sm.short_on) {
        float mw = CSD_NEG_INF;
        for (int i = lane; i < wcp; i += 32) mw = max_nan(mw, sm.list[warp][i]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mw = max_nan(mw, __shfl_xor_sync(0xffffffffu, mw, off));
        const float hi = lo + a.hi_delta * dev;
        const float ztok = r < kBlockRows ? sm.rs.tokz[r] : 0.0f;
        float acc = 0.0f;
        int cmax = 0, cgt = 0, rk = 0;
        for (int i = lane; i < wcp; i += 32) {
          const float v = sm.list[warp][i];
          const float ev = ex2f((v - mw) * kLog2e);   // (0 for the padding)
          acc += (v != mw) ? ev : 0.0f;
          cmax += (v == mw) ? 1 : 0;
          cgt += (v > hi) ? 1 : 0;
          rk += (v > ztok) ? 1 : 0;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        cmax = __reduce_add_sync(0xffffffffu, cmax);
        cgt = __reduce_add_sync(0xffffffffu, cgt);
        rk = __reduce_add_sync(0xffffffffu, rk);
        int last_s = 0;
        if (lane == 0) {
          sm.fw_m[warp] = mw;
          sm.fw_s[warp] = wcp > 0 ? acc + (float)(cmax - 1) : -1.0f;   // (an empty list: the identity)
          sm.fw_cgt[warp] = cgt;
          sm.fw_rk[warp] = rk;
          __threadfence_block();
          last_s = atom_add_shared(&sm.arrive[0], 1) == kTopkWarps - 1 ? 1 : 0;
        }
        last_s = __shfl_sync(0xffffffffu, last_s, 0);
        if (last_s) {
          if (lane == 0) sm.arrive[0] = 0;
          __threadfence_block();
          const bool mine = lane < kTopkWarps;
          float m = mine ? sm.fw_m[lane] : CSD_NEG_INF, sv = mine ? sm.fw_s[lane] : -1.0f;
          int n_lo = mine ? sm.wpos[lane] : 0;
          const bool over = __any_sync(0xffffffffu, n_lo > WL);
          const bool nan_m = __any_sync(0xffffffffu, m != m);
          n_lo = __reduce_add_sync(0xffffffffu, n_lo);
          const int cg = __reduce_add_sync(0xffffffffu, mine ? sm.fw_cgt[lane] : 0);
          const int rank = __reduce_add_sync(0xffffffffu, mine ? sm.fw_rk[lane] : 0);
#pragma unroll
          for (int off = 4; off > 0; off >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m, off), s2 = __shfl_xor_sync(0xffffffffu, sv, off);
            stat_merge(m, sv, m2, s2);
          }
          if (lane == 0) {
            // bound on what the filter removes: at least k of the gathered values are kept, and with fewer than k
            // values above hi every one it removes lies at or below hi
            const float dropped = (float)(n_lo - k_top) * ex2f((hi - m) * kLog2e);
            const bool ok = !over && !nan_m && n_lo >= k_top && cg < k_top && m > lo && m < CSD_POS_INF &&
                            sv >= 0.0f && sv < CSD_POS_INF && dropped <= 1.4901161e-8f;
            if (ok && r < kBlockRows) {
              sm.rs.ms[r] = make_float2(m, sv);
              sm.rs.thr[r] = lo;
              if (!(rank < k_top)) sm.rs.tokz[r] = CSD_NEG_INF;   // the exact filter drops the drafted token
            }
            // (a single row can fail -- a row maximum on the low side leaves the bound short -- without the
            // next ones doing so; rows that are flat keep failing, and after three such the block stops trying)
            if (!ok && ++sm.short_fail >= 3) sm.short_on = 0;
            sm.row_short = ok ? 1 : 0;
          }
        }
        __syncthreads();   // ---- D: settled, or on to the full selection
        if (sm.row_short) continue;
      }
      float mx = CSD_NEG_INF;
      for (int i = lane; i < wcp; i += 32) {
        const float v = sm.list[warp][i];
        mx = max_nan(mx, v);
        const int bv = lin_bin(v, lo, scale);   // (the padding gets a negative bin)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ge.s32 p, %1, 0;\n\t@p red.shared.add.u32 [%0], 1;\n\t}"
                     ::"r"(hist_addr + 4u * (uint32_t)bv), "r"(bv)
                     : "memory");
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = max_nan(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      __syncwarp();
      int last = 0;
      if (lane == 0) {
        sm.wmax[warp] = mx;
        __threadfence_block();
        last = atom_add_shared(&sm.arrive[0], 1) == kTopkWarps - 1 ? 1 : 0;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        // The last warp to get here decides for the row: can the lists be used, and if so, which bin
        // holds the k-th largest and which rank the answer has inside it.
        if (lane == 0) sm.arrive[0] = 0;
        __threadfence_block();
        int n_lo = 0;
        bool fast = true;
        float m = sm.wmax[0];
#pragma unroll
        for (int w = 0; w < kTopkWarps; ++w) {
          const int cw = sm.wpos[w];
          if (cw > WL) fast = false;
          n_lo += cw;
          m = max_nan(m, sm.wmax[w]);
        }
        // NaN guesses, NaN / +inf rows and constant rows all fail one of these tests
        fast = fast && n_lo >= k_top && (m > lo) && (m < CSD_POS_INF) && (scale > 0.0f) && (scale < CSD_POS_INF);
        if (fast) {
          int kk;
          const int bin = warp_pick_bin(sm.hist, k_top, lane, &kk);
          if (lane == 0) { sm.bc_i[0] = bin; sm.bc_i[1] = kk; }
        }
        if (lane == 0) {
          // a guess that missed moves the next one of this kind of row: down if too few values were
          // gathered, up if a list overflowed (a NaN multiplier -- no guess at all -- stays NaN)
          if (!fast && n_lo < k_top) { sm.c_kind[par] -= 0.5f; sm.adapt_on = 1; }
          else if (!fast && n_lo > kListCap / 2) { sm.c_kind[par] += 0.35f; sm.adapt_on = 1; }
          sm.row_mx = m;
          sm.row_fast = fast ? 1 : 0;
          if (!fast && r < kBlockRows) atomicOr(&sm.need_exact[r >> 5], 1u << (r & 31));
        }
      }
      __syncthreads();   // ---- C: decision and bin known
      if (!sm.row_fast) continue;   // selected exactly after the loop
      mx = sm.row_mx;
      {
        // ---- second pass: statistics of the values above the bin; the bin's own values are set aside
        const int pick_bin = sm.bc_i[0];
        float acc = 0.0f;
        int cmax = 0;
        for (int i = lane; i < wcp; i += 32) {
          const float v = sm.list[warp][i];
          const int bv = lin_bin(v, lo, scale);   // (-inf, the padding, is below every bin)
          const float ev = ex2f((v - mx) * kLog2e);
          const bool above = bv > pick_bin;
          acc += (above && v != mx) ? ev : 0.0f;
          cmax += (above && v == mx) ? 1 : 0;
          if (bv == pick_bin) {
            const int slot = atomicAdd(&sm.n_cand[par], 1);
            if (slot < kCandCap) sm.cand[slot] = v;
          }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          acc += __shfl_xor_sync(0xffffffffu, acc, off);
          cmax += __shfl_xor_sync(0xffffffffu, cmax, off);
        }
        __syncwarp();
        last = 0;
        if (lane == 0) {
          sm.part_acc[par][warp] = acc;
          sm.part_cmax[par][warp] = cmax;
          __threadfence_block();
          last = atom_add_shared(&sm.arrive[1], 1) == kTopkWarps - 1 ? 1 : 0;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          // The last warp to get here ranks the bin's values exactly (two per lane): the threshold is
          // the one of rank kk from the top; those not below it join the statistics.  The other warps
          // have gone on to the next row; its first barrier orders these results before their use.
          if (lane == 0) sm.arrive[1] = 0;
          __threadfence_block();
          const int n_cand = sm.n_cand[par];
          if (n_cand <= kCandCap) {
            const int kk = sm.bc_i[1];
            const float v0 = lane < n_cand ? sm.cand[lane] : CSD_NEG_INF;
            const float v1 = lane + 32 < n_cand ? sm.cand[lane + 32] : CSD_NEG_INF;
            int gt0 = 0, ge0 = 0, gt1 = 0, ge1 = 0;
            for (int j2 = 0; j2 < n_cand; ++j2) {
              const float w = sm.cand[j2];
              gt0 += (w > v0) ? 1 : 0; ge0 += (w >= v0) ? 1 : 0;
              gt1 += (w > v1) ? 1 : 0; ge1 += (w >= v1) ? 1 : 0;
            }
            const bool hit0 = lane < n_cand && gt0 < kk && kk <= ge0;
            const bool hit1 = lane + 32 < n_cand && gt1 < kk && kk <= ge1;
            const unsigned b0 = __ballot_sync(0xffffffffu, hit0);
            const unsigned b1 = __ballot_sync(0xffffffffu, hit1);
            const float thr = b0 ? __shfl_sync(0xffffffffu, v0, __ffs(b0) - 1)
                                 : __shfl_sync(0xffffffffu, v1, b1 ? __ffs(b1) - 1 : 0);
            float acc2 = 0.0f;
            int cmax2 = 0;
            if (lane < n_cand && v0 >= thr) { if (v0 == mx) cmax2 += 1; else acc2 += ex2f((v0 - mx) * kLog2e); }
            if (lane + 32 < n_cand && v1 >= thr) { if (v1 == mx) cmax2 += 1; else acc2 += ex2f((v1 - mx) * kLog2e); }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
              acc2 += __shfl_xor_sync(0xffffffffu, acc2, off);
              cmax2 += __shfl_xor_sync(0xffffffffu, cmax2, off);
            }
            if (lane == 0) {
              // every warp published its partials before it counted itself in: the row is complete
              float tot = acc2;
              int ctot = cmax2;
#pragma unroll
              for (int w = 0; w < kTopkWarps; ++w) { tot += sm.part_acc[par][w]; ctot += sm.part_cmax[par][w]; }
              if (r < kBlockRows) {
                sm.rs.ms[r] = make_float2(mx, tot + (float)(ctot - 1));
                sm.rs.thr[r] = thr;
              }
              // where the threshold really sat, in deviations from the mean: the next row of this kind
              // guesses a little below that (half-way from the current multiplier)
              // (only once the plain guess has missed in this block: data it fits is left alone)
              if (sm.adapt_on) {
                const float c_seen = (thr - sm.row_mean[par]) / sm.row_dev[par] + a.lo_delta;
                if (c_seen == c_seen && fabsf(c_seen) < 64.0f) sm.c_kind[par] = 0.5f * (sm.c_kind[par] + c_seen);
              }
            }
          } else if (lane == 0 && r < kBlockRows) {   // crowded bin
            atomicOr(&sm.need_exact[r >> 5], 1u << (r & 31));
          }
        }
      }
    }
    // ---- rows whose lists could not be used: exact select and statistics from global memory (rare) ----
    __syncthreads();
    for (int r = 0; r < n_rows && r < kBlockRows; ++r) {
      if (((sm.need_exact[r >> 5] >> (r & 31)) & 1u) == 0u) continue;   // the same decision in every thread
      float m_e = 0.0f, s_e = 0.0f, thr_e = 0.0f;
      exact_row_from_global<T, CFG, Smem>(row_of(r), V, k_top, sm, tid, m_e, s_e, thr_e);
      if (tid == 0) {
        sm.rs.ms[r] = make_float2(m_e, s_e);
        sm.rs.thr[r] = thr_e;
      }
    }
    if (sm.abort && tid == 0) {
      if (a.error_flag) atomicExch(a.error_flag, 1);
      // Nothing was issued after the first failed wait was seen, so the copies that may still be in
      // flight are those of chunks [waited, issued_q): at most one per stage.  Wait for each, bounded.
      for (int c = waited; c < sm.issued_q; ++c)
        (void)mbar_wait(&sm.full[c & 1], (uint32_t)(c >> 1) & 1u, a.wait_limit);
    }
  }

  // ================================= phase 2 ===========================================
  __syncthreads();
  if (stats_only) {
    write_row_stats(a, sh, sm.rs, tid, kTopkThreads, sm.abort != 0);
    return;
  }
  static_assert(sizeof(sm.list) >= kFinTiles * sizeof(double), "tile sums live in the list area");
  finish_block<T, CFG, kTopkThreads, true>(a, sh, sm.rs, tid, sm.abort != 0, &sm.ring[0][0], kTkRingBytes,
                                     reinterpret_cast<double*>(&sm.list[0][0]), sm.fin, sm.fst);
}

}  // namespace csd
