// Device code of libcsd: the verify-and-resample round of Cool-SD on sm_100a.
//
// Two kernels per call (three with top-k filtering), the last launched with
// programmatic dependent launch so that its blocks are resident and waiting
// when the statistics kernel drains:
//
//   topk_threshold_kernel  (top-k only) exact k-th largest value of every row by
//                      radix select; the value is the filter threshold.
//   row_stats_kernel   streams every logit row once from HBM (the only HBM
//                      traffic of the call) and leaves, per (row, part), the pair
//                      (m, s) with  sum_x exp(z_x) = (1 + s) * exp(m)  over that part:
//                      m the maximum, s the sum of exp(z - m) over all OTHER
//                      entries.  Keeping the "1 +" out of the fp32 sum preserves the
//                      relative accuracy of 1 - P(argmax) on sharply peaked rows.
//   finish_kernel      one block per sequence: merges the parts, gathers the
//                      drafted tokens' logits, evaluates Eq. relax and the accept
//                      tests, finds tau, re-reads the two rows of position tau+1
//                      (L2 hits at the sizes of interest), forms Eq. opt_G, and
//                      draws by inverse CDF with fp64 running sums.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace csd {

constexpr int kStatsThreads = 256;
constexpr int kFinishThreads = 1024;
constexpr int kMaxGamma = 32;
constexpr float kLog2e = 1.4426950408889634f;
#define CSD_NEG_INF (__int_as_float(0xff800000))
#define CSD_POS_INF (__int_as_float(0x7f800000))

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- (m, s) algebra ---------------------------------------------------------
// identity: m = -inf, s = -1 (so that 1 + s = 0)
__device__ __forceinline__ void stat_merge(float& m, float& s, float m2, float s2) {
  if (m2 > m) {
    float t = m; m = m2; m2 = t;
    t = s; s = s2; s2 = t;
  }
  if (m2 != CSD_NEG_INF) s += (1.0f + s2) * ex2f((m2 - m) * kLog2e);
}

__device__ __forceinline__ void stat_warp_allreduce(float& m, float& s) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    float s2 = __shfl_xor_sync(0xffffffffu, s, off);
    stat_merge(m, s, m2, s2);
  }
}

// (m, s) of n register-resident values
template <int N>
__device__ __forceinline__ void stat_of_values(const float (&z)[N], float& m, float& s) {
  m = CSD_NEG_INF;
#pragma unroll
  for (int k = 0; k < N; ++k) m = fmaxf(m, z[k]);
  float acc = 0.0f;
  int cnt = 0;
#pragma unroll
  for (int k = 0; k < N; ++k) {
    float e = ex2f((z[k] - m) * kLog2e);
    if (z[k] == m) cnt += 1; else acc += e;   // NaN entries poison acc, which marks the row
  }
  s = acc + (float)(cnt - 1);
}

// ---- element access -----------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;
  __device__ static __forceinline__ void load_vec(const float* p, float (&out)[4]) {
    float4 v = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
  __device__ static __forceinline__ float load_one(const float* p) { return __ldg(p); }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static __forceinline__ void load_vec(const __nv_bfloat16* p, float (&out)[8]) {
    uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      out[2 * k] = __uint_as_float(w[k] << 16);
      out[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ float load_one(const __nv_bfloat16* p) {
    return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
  }
};

// guidance mix: the difference is rounded to fp32, then one fused multiply-add
__device__ __forceinline__ float cfg_mix(float c, float u, float s) {
  return __fmaf_rn(s, __fsub_rn(c, u), u);
}

// One logical row: conditional array, optional unconditional array, optional
// top-k threshold.  Loads VEC consecutive logits starting at element x0.
template <typename T, bool CFG>
struct Row {
  const T* cond;
  const T* uncond;
  float scale;
  float thr;  // entries below thr become -inf (thr = -inf: no filter)
  static constexpr int kVec = Elem<T>::kVec;

  __device__ __forceinline__ void load_vec(int x0, float (&z)[Elem<T>::kVec]) const {
    Elem<T>::load_vec(cond + x0, z);
    if (CFG) {
      float u[kVec];
      Elem<T>::load_vec(uncond + x0, u);
#pragma unroll
      for (int k = 0; k < kVec; ++k) z[k] = cfg_mix(z[k], u[k], scale);
    }
  }
  __device__ __forceinline__ float load_one(int x) const {
    float z = Elem<T>::load_one(cond + x);
    if (CFG) z = cfg_mix(z, Elem<T>::load_one(uncond + x), scale);
    return z;
  }
  // vector when allowed, otherwise bounds-checked scalars; out-of-range -> -inf
  __device__ __forceinline__ void load_tile(int x0, int V, bool vec_ok, float (&z)[Elem<T>::kVec]) const {
    if (vec_ok) {
      if (x0 < V) load_vec(x0, z);
      else {
#pragma unroll
        for (int k = 0; k < kVec; ++k) z[k] = CSD_NEG_INF;
      }
    } else {
#pragma unroll
      for (int k = 0; k < kVec; ++k) z[k] = (x0 + k < V) ? load_one(x0 + k) : CSD_NEG_INF;
    }
  }
  __device__ __forceinline__ float filter(float z) const { return z < thr ? CSD_NEG_INF : z; }
};

// ============================ kernel 1: row statistics ==========================
struct StatsArgs {
  const void* target;
  const void* draft;
  const void* target_uncond;
  const void* draft_uncond;
  float cfg_scale;
  int B, gamma, T, V;
  int64_t tstride, dstride;  // elements
  int parts;                 // parts per row
  int part_elems;            // elements per part (multiple of the vector width)
  int n_items;               // B * (T + gamma) * parts
  int vec_ok;
  float2* partials;          // [B * (T + gamma)][parts]
  const float* thresholds;   // [B * (T + gamma)], read only by the TOPK variants
};

// U = 16-byte loads per thread per array per item
template <typename T, bool CFG, int U, bool TOPK>
__global__ void __launch_bounds__(kStatsThreads) row_stats_kernel(const StatsArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  __shared__ float sh_m[2][kStatsThreads / 32];
  __shared__ float sh_s[2][kStatsThreads / 32];
  pdl_launch_dependents();  // the finishing kernel may become resident as soon as blocks retire

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rows_per_seq = a.T + a.gamma;
  int buf = 0;
  for (int item = blockIdx.x; item < a.n_items; item += gridDim.x, buf ^= 1) {
    const int part = item % a.parts;
    const int row_id = item / a.parts;
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    Row<T, CFG> row;
    row.scale = a.cfg_scale;
    row.thr = TOPK ? a.thresholds[row_id] : CSD_NEG_INF;
    if (r < a.T) {
      const int64_t off = (int64_t)b * a.tstride + (int64_t)r * a.V;
      row.cond = reinterpret_cast<const T*>(a.target) + off;
      row.uncond = CFG ? reinterpret_cast<const T*>(a.target_uncond) + off : nullptr;
    } else {
      const int64_t off = (int64_t)b * a.dstride + (int64_t)(r - a.T) * a.V;
      row.cond = reinterpret_cast<const T*>(a.draft) + off;
      row.uncond = CFG ? reinterpret_cast<const T*>(a.draft_uncond) + off : nullptr;
    }
    const int x_begin = part * a.part_elems;
    const int x_end = min(a.V, x_begin + a.part_elems);

    float m, s;
    if (a.vec_ok) {
      float z[U][VEC];
#pragma unroll
      for (int k = 0; k < U; ++k) {
        const int x0 = x_begin + (k * kStatsThreads + tid) * VEC;
        if (x0 < x_end) {
          row.load_vec(x0, z[k]);
          if (TOPK) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) z[k][e] = row.filter(z[k][e]);
          }
        } else {
#pragma unroll
          for (int e = 0; e < VEC; ++e) z[k][e] = CSD_NEG_INF;
        }
      }
      // all loads are in flight before the first use
      float flat[U * VEC];
#pragma unroll
      for (int k = 0; k < U; ++k)
#pragma unroll
        for (int e = 0; e < VEC; ++e) flat[k * VEC + e] = z[k][e];
      stat_of_values(flat, m, s);
      // a thread whose slots were all padding reports the identity
      // (padding entries are -inf and contribute exp(-inf) = 0 next to real values)
      if (x_begin + tid * VEC >= x_end) { m = CSD_NEG_INF; s = -1.0f; }
    } else {
      m = CSD_NEG_INF; s = -1.0f;
      for (int x = x_begin + tid; x < x_end; x += kStatsThreads) {
        float one[1] = {TOPK ? row.filter(row.load_one(x)) : row.load_one(x)};
        float m1, s1;
        stat_of_values(one, m1, s1);
        stat_merge(m, s, m1, s1);
      }
    }
    stat_warp_allreduce(m, s);
    if (lane == 0) { sh_m[buf][warp] = m; sh_s[buf][warp] = s; }
    __syncthreads();
    if (warp == 0) {
      float mm = lane < kStatsThreads / 32 ? sh_m[buf][lane] : CSD_NEG_INF;
      float ss = lane < kStatsThreads / 32 ? sh_s[buf][lane] : -1.0f;
#pragma unroll
      for (int off = kStatsThreads / 64; off > 0; off >>= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, mm, off);
        float s2 = __shfl_xor_sync(0xffffffffu, ss, off);
        stat_merge(mm, ss, m2, s2);
      }
      if (lane == 0) a.partials[(int64_t)row_id * a.parts + part] = make_float2(mm, ss);
    }
    // double-buffered staging: the next item writes the other buffer, and the
    // barrier of that item orders this item's reads before the buffer's reuse
  }
}


// ============================ kernel 0: top-k thresholds (any V) ===================
// Exact k-th largest value of every (mixed) row by a most-significant-digit-first
// radix select over order-preserving 32-bit keys: three passes over the row with
// digits of 11, 11 and 10 bits.  The value itself is the threshold, so ties with
// the k-th largest are kept whatever their position.
constexpr int kSelectThreads = 1024;
constexpr int kSelectBins = 2048;

__device__ __forceinline__ uint32_t order_key(float z) {
  const uint32_t b = __float_as_uint(z);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_value(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

struct SelectArgs {
  const void* target;
  const void* draft;
  const void* target_uncond;
  const void* draft_uncond;
  float cfg_scale;
  int B, gamma, T, V;
  int64_t tstride, dstride;
  int vec_ok;
  int top_k;          // 1 <= top_k < V
  float* thresholds;  // [B * (T + gamma)]
};

// Walks a histogram from its top bin down and returns the bin that holds the
// k-th largest key; *above gets the number of keys in higher bins.  One warp.
__device__ __forceinline__ int select_bin_from_top(const int* hist, int nbins, int k, int lane, int* above) {
  const int chunk = nbins / 32;                     // nbins is a multiple of 32
  const int hi = nbins - lane * chunk;              // lane 0 owns the top chunk
  int local = 0;
  for (int d = hi - 1; d >= hi - chunk; --d) local += hist[d];
  int incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  const unsigned ballot = __ballot_sync(0xffffffffu, incl >= k);
  const int owner = ballot ? __ffs(ballot) - 1 : 31;  // fewer than k keys: the lowest chunk
  int bin = 0, cnt_above = 0;
  if (lane == owner) {
    int c = incl - local;
    bin = hi - chunk;
    cnt_above = c;
    for (int d = hi - 1; d >= hi - chunk; --d) {
      if (c + hist[d] >= k) { bin = d; cnt_above = c; break; }
      c += hist[d];
      cnt_above = c;
    }
  }
  bin = __shfl_sync(0xffffffffu, bin, owner);
  *above = __shfl_sync(0xffffffffu, cnt_above, owner);
  return bin;
}

template <typename T, bool CFG>
__global__ void __launch_bounds__(kSelectThreads) topk_threshold_kernel(const SelectArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  __shared__ int hist[kSelectBins];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_k;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rows_per_seq = a.T + a.gamma;
  const int n_rows = a.B * rows_per_seq;
  for (int row_id = blockIdx.x; row_id < n_rows; row_id += gridDim.x) {
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    Row<T, CFG> row;
    row.scale = a.cfg_scale;
    row.thr = CSD_NEG_INF;
    if (r < a.T) {
      const int64_t off = (int64_t)b * a.tstride + (int64_t)r * a.V;
      row.cond = reinterpret_cast<const T*>(a.target) + off;
      row.uncond = CFG ? reinterpret_cast<const T*>(a.target_uncond) + off : nullptr;
    } else {
      const int64_t off = (int64_t)b * a.dstride + (int64_t)(r - a.T) * a.V;
      row.cond = reinterpret_cast<const T*>(a.draft) + off;
      row.uncond = CFG ? reinterpret_cast<const T*>(a.draft_uncond) + off : nullptr;
    }
    uint32_t prefix = 0, mask = 0;
    int k = a.top_k;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const int nbins = pass == 2 ? 1024 : 2048;
      for (int d = tid; d < nbins; d += kSelectThreads) hist[d] = 0;
      __syncthreads();
      for (int x0 = tid * VEC; x0 < a.V; x0 += kSelectThreads * VEC) {
        float z[VEC];
        row.load_tile(x0, a.V, a.vec_ok, z);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          const uint32_t key = order_key(z[e]);
          if (x0 + e < a.V && (key & mask) == prefix) atomicAdd(&hist[(key >> shift) & (nbins - 1)], 1);
        }
      }
      __syncthreads();
      if (warp == 0) {
        int above;
        const int bin = select_bin_from_top(hist, nbins, k, lane, &above);
        if (lane == 0) {
          sh_prefix = prefix | ((uint32_t)bin << shift);
          sh_k = k - above;
        }
      }
      __syncthreads();
      prefix = sh_prefix;
      k = sh_k;
      mask |= (uint32_t)(nbins - 1) << shift;
    }
    if (tid == 0) a.thresholds[row_id] = order_value(prefix);
    __syncthreads();
  }
}

// ============================ kernel 2: per-sequence finish =====================
struct FinishArgs {
  const void* target;
  const void* draft;
  const void* target_uncond;
  const void* draft_uncond;
  float cfg_scale;
  int B, gamma, T, V;
  int64_t tstride, dstride;
  int parts;
  int vec_ok;
  int use_topk;
  const float2* partials;   // [B*(T+gamma)][parts]
  const float* thresholds;  // [B*(T+gamma)] (top-k only)
  const int32_t* tokens;
  const float* uniforms;
  const float* schedule;
  int32_t* out_tokens;
  int32_t* out_accept_len;
  int32_t* out_status;
  float* dbg_p;
  float* dbg_q;
  float* dbg_f;
  float* dbg_G;
};

struct PairCtx {  // what Eq. opt_G needs at one position
  float Mt, St, Md, Sd;   // (m, s) of the target and drafter rows
  float inv_t;            // 1 / (1 + St)
  float inv_den;          // 1 / ((1 + St)(1 + Sd))
  float one_minus_omega;
  int mode;               // 0: Eq. opt_G; 1: weights = P (bonus draw, unusable drafter row, Z fallback)
};

// unnormalised weight of one candidate token.  P - Q is formed as
// ((et - ed) + (et*Sd - ed*St)) / ((1+St)(1+Sd)), which has no cancellation
// beyond that of the inputs when both rows peak on the same token.
__device__ __forceinline__ float weight_of(float zt, float zd, const PairCtx& c) {
  const float et = ex2f((zt - c.Mt) * kLog2e);
  if (c.mode == 1) return et * c.inv_t;
  const float ed = ex2f((zd - c.Md) * kLog2e);
  const float pq = ((et - ed) + (et * c.Sd - ed * c.St)) * c.inv_den;  // P - Q
  const float alt = c.one_minus_omega * et * c.inv_t;                    // (1 - omega) P
  return fmaxf(0.0f, fmaxf(pq, alt));
}

__device__ __forceinline__ double warp_sum_double(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}
__device__ __forceinline__ double warp_incl_scan_double(double v, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    double t = __shfl_up_sync(0xffffffffu, v, off);
    if (lane >= off) v += t;
  }
  return v;
}

// Shared-memory state of one sequence's finish.
struct FinishSmem {
  float M[2][kMaxGamma + 1], S[2][kMaxGamma + 1], thr[2][kMaxGamma + 1];
  int acc[kMaxGamma], flag[kMaxGamma + 1], valid[2][kMaxGamma + 1];
  int pick_tile;
  int token;
  double pick_prefix, Z;
};

// Barrier over the NT threads that run the finish: the whole block (BAR == 0) or
// a named barrier when other warps of the block do not take part.
template <int NT, int BAR>
__device__ __forceinline__ void group_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// Everything after the row statistics for sequence b, run by NT threads (tid in
// [0, NT)): merge the parts, Eq. relax and the accept tests, tau, Eq. opt_G at
// position tau+1, the inverse-CDF draw, the emitted block.  tile_sums needs one
// double per tile of 32 * (16 bytes / element size) tokens.
template <typename T, bool CFG, int NT, int BAR>
__device__ void finish_sequence(const FinishArgs& a, const int b, const int tid, double* tile_sums,
                                FinishSmem& sm, const int extra_status) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  const int lane = tid & 31, warp = tid >> 5;
  const int L = a.gamma, V = a.V;
  const int rows_per_seq = a.T + L;
  const T* tgt = reinterpret_cast<const T*>(a.target) + (int64_t)b * a.tstride;
  const T* dft = reinterpret_cast<const T*>(a.draft) + (int64_t)b * a.dstride;
  const T* tgt_u = CFG ? reinterpret_cast<const T*>(a.target_uncond) + (int64_t)b * a.tstride : nullptr;
  const T* dft_u = CFG ? reinterpret_cast<const T*>(a.draft_uncond) + (int64_t)b * a.dstride : nullptr;

  // ---- 1. per position: merge parts, gather, Eq. relax, accept test ------------
  for (int i = warp; i <= L; i += NT / 32) {
    const bool has_t = i < a.T, has_d = i < L;
    float M[2] = {CSD_NEG_INF, CSD_NEG_INF}, S[2] = {-1.0f, -1.0f};
    float thr[2] = {CSD_NEG_INF, CSD_NEG_INF};
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      if (which == 0 ? !has_t : !has_d) continue;
      const int64_t row_id = (int64_t)b * rows_per_seq + (which == 0 ? i : a.T + i);
      float m = CSD_NEG_INF, s = -1.0f;
      for (int p = lane; p < a.parts; p += 32) {
        const float2 v = __ldcg(a.partials + row_id * a.parts + p);
        stat_merge(m, s, v.x, v.y);
      }
      stat_warp_allreduce(m, s);
      M[which] = m; S[which] = s;
      if (a.use_topk) thr[which] = __ldcg(a.thresholds + row_id);
    }
    if (lane == 0) {
      const bool t_ok = has_t && M[0] > CSD_NEG_INF && M[0] < CSD_POS_INF && S[0] >= 0.0f && S[0] < CSD_POS_INF;
      const bool d_ok = has_d && M[1] > CSD_NEG_INF && M[1] < CSD_POS_INF && S[1] >= 0.0f && S[1] < CSD_POS_INF;
      sm.M[0][i] = M[0]; sm.S[0][i] = S[0]; sm.thr[0][i] = thr[0];
      sm.M[1][i] = M[1]; sm.S[1][i] = S[1]; sm.thr[1][i] = thr[1];
      sm.valid[0][i] = t_ok; sm.valid[1][i] = d_ok;
      int flag = 0;
      if (i < L) {
        const int tok = a.tokens[(int64_t)b * L + i];
        const bool tok_ok = tok >= 0 && tok < V;
        float omega = a.schedule[i];
        omega = omega >= 0.0f ? omega : 0.0f;
        float f = 0.0f, p = __int_as_float(0x7fc00000), q = p;
        if (!t_ok || !d_ok) flag = 1;
        else if (!tok_ok) flag = 2;
        else {
          Row<T, CFG> rt{tgt + (int64_t)i * V, CFG ? tgt_u + (int64_t)i * V : nullptr, a.cfg_scale, thr[0]};
          Row<T, CFG> rd{dft + (int64_t)i * V, CFG ? dft_u + (int64_t)i * V : nullptr, a.cfg_scale, thr[1]};
          const float dt = rt.filter(rt.load_one(tok)) - M[0];
          const float dd = rd.filter(rd.load_one(tok)) - M[1];
          p = ex2f(dt * kLog2e) / (1.0f + S[0]);
          q = ex2f(dd * kLog2e) / (1.0f + S[1]);
          if (dd == CSD_NEG_INF) f = 1.0f;         // q = 0: p/q = +inf, and 0/0 := 1
          else if (dt == CSD_NEG_INF) f = 0.0f;    // p = 0 < q
          else f = fminf(1.0f, omega * ex2f((dt - dd) * kLog2e) * ((1.0f + S[1]) / (1.0f + S[0])));
        }
        const float r = a.uniforms[(int64_t)b * (L + 1) + i];
        sm.acc[i] = (r <= f) ? 1 : 0;
        if (a.dbg_p) a.dbg_p[(int64_t)b * L + i] = p;
        if (a.dbg_q) a.dbg_q[(int64_t)b * L + i] = q;
        if (a.dbg_f) a.dbg_f[(int64_t)b * L + i] = f;
      }
      sm.flag[i] = flag;
    }
  }
  group_sync<NT, BAR>();

  // ---- 2. tau = number of leading accepts (the for/break of Algorithm 1) --------
  int tau = 0;
  while (tau < L && sm.acc[tau]) ++tau;
  int status = extra_status;
  for (int i = 0; i <= min(tau, L - 1); ++i) status |= sm.flag[i];

  // ---- 3. which row to draw from -------------------------------------------------
  const int j = tau;  // 0-based row index of position tau+1 (j == L: bonus row)
  PairCtx ctx;
  bool draw = true;
  if (j < L) {
    if (!sm.valid[0][j]) draw = false;
    ctx.mode = sm.valid[1][j] ? 0 : 1;
  } else {
    if (a.T == L + 1) {
      ctx.mode = 1;
      if (!sm.valid[0][L]) { draw = false; status |= 1; }
    } else draw = false;
  }
  float* G_out = a.dbg_G ? a.dbg_G + (int64_t)b * V : nullptr;
  const int ntiles = (V + TILE - 1) / TILE;
  int token = -1;

  if (draw) {
    ctx.Mt = sm.M[0][j]; ctx.St = sm.S[0][j];
    ctx.Md = j < L ? sm.M[1][j] : 0.0f; ctx.Sd = j < L ? sm.S[1][j] : 0.0f;
    ctx.inv_t = 1.0f / (1.0f + ctx.St);
    ctx.inv_den = ctx.inv_t / (1.0f + ctx.Sd);
    float omega = j < L ? a.schedule[j] : 0.0f;
    omega = omega >= 0.0f ? omega : 0.0f;
    ctx.one_minus_omega = 1.0f - omega;
    Row<T, CFG> rt{tgt + (int64_t)j * V, CFG ? tgt_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[0][j]};
    Row<T, CFG> rd = rt;
    if (j < L) rd = Row<T, CFG>{dft + (int64_t)j * V, CFG ? dft_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[1][j]};
    const float u = a.uniforms[(int64_t)b * (L + 1) + L];

    for (int attempt = 0; attempt < 2; ++attempt) {
      // ---- 4. Eq. opt_G weights, one fp64 sum per tile ---------------------------
      // several tiles per warp and trip (registers permitting), all loads issued before the first use
      constexpr int UNR = NT > 256 ? 1 : 16 / VEC;
      for (int tile0 = warp; tile0 < ntiles; tile0 += UNR * (NT / 32)) {
        float zt[UNR][VEC], zd[UNR][VEC];
#pragma unroll
        for (int r = 0; r < UNR; ++r) {
          const int tile = tile0 + r * (NT / 32);
          const int x0 = tile * TILE + lane * VEC;
          if (tile < ntiles) {
            rt.load_tile(x0, V, a.vec_ok, zt[r]);
            if (ctx.mode == 0) rd.load_tile(x0, V, a.vec_ok, zd[r]);
          }
        }
#pragma unroll
        for (int r = 0; r < UNR; ++r) {
          const int tile = tile0 + r * (NT / 32);
          if (tile < ntiles) {
            float acc = 0.0f;
#pragma unroll
            for (int k = 0; k < VEC; ++k)
              acc += weight_of(rt.filter(zt[r][k]), ctx.mode == 0 ? rd.filter(zd[r][k]) : 0.0f, ctx);
            const double tsum = warp_sum_double((double)acc);
            if (lane == 0) tile_sums[tile] = tsum;
          }
        }
      }
      group_sync<NT, BAR>();
      // ---- 5. locate the tile that holds the crossing C(x) > u Z ------------------
      if (warp == 0) {
        const int chunk = (ntiles + 31) / 32;
        const int t0 = lane * chunk, t1 = min(ntiles, t0 + chunk);
        double local = 0.0;
        for (int t = t0; t < t1; ++t) local += tile_sums[t];
        const double incl = warp_incl_scan_double(local, lane);
        const double Z = __shfl_sync(0xffffffffu, incl, 31);
        const double target = (double)u * Z;
        const bool mine = incl > target && local > 0.0;
        const unsigned ballot = __ballot_sync(0xffffffffu, mine);
        if (lane == 0) { sm.Z = Z; sm.pick_tile = -1; }
        __syncwarp();
        if (ballot != 0 && lane == __ffs(ballot) - 1) {
          double c = incl - local, c_pick = c;
          int pick = t0;
          for (int t = t0; t < t1; ++t) {
            const double v = tile_sums[t];
            if (v > 0.0) { pick = t; c_pick = c; }   // last tile with mass seen so far
            if (c + v > target && v > 0.0) break;
            c += v;
          }
          sm.pick_tile = pick;
          sm.pick_prefix = c_pick;
        }
      }
      group_sync<NT, BAR>();
      const double Z = sm.Z;
      if (!(Z > 0.0) || !(Z < (double)CSD_POS_INF)) {
        if (attempt == 0 && ctx.mode == 0) {  // empty positive part: fall back to G := P_j
          ctx.mode = 1;
          status |= 4;
          group_sync<NT, BAR>();
          continue;
        }
        break;  // nothing to draw from
      }
      // ---- 6. scan inside that tile -------------------------------------------------
      if (warp == 0) {
        const int tile = sm.pick_tile;
        const double target = (double)u * Z;
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC], zd[VEC];
        rt.load_tile(x0, V, a.vec_ok, zt);
        if (ctx.mode == 0) rd.load_tile(x0, V, a.vec_ok, zd);
        double run[VEC];
        double acc = 0.0;
        int last_pos = -1;
        unsigned posmask = 0;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          const float g = weight_of(rt.filter(zt[k]), ctx.mode == 0 ? rd.filter(zd[k]) : 0.0f, ctx);
          if (g > 0.0f) { last_pos = k; posmask |= 1u << k; }
          acc += (double)g;
          run[k] = acc;
        }
        const double before = sm.pick_prefix + (warp_incl_scan_double(acc, lane) - acc);
        int first = -1;
#pragma unroll
        for (int k = VEC - 1; k >= 0; --k)
          if (before + run[k] > target && ((posmask >> k) & 1u)) first = k;
        const unsigned hit = __ballot_sync(0xffffffffu, first >= 0);
        const unsigned pos = __ballot_sync(0xffffffffu, last_pos >= 0);
        if (hit != 0) {
          if (lane == __ffs(hit) - 1) sm.token = x0 + first;
        } else if (pos != 0) {  // rounding left no crossing: last token with positive weight
          if (lane == 31 - __clz(pos)) sm.token = x0 + last_pos;
        } else if (lane == 0) sm.token = -1;
      }
      group_sync<NT, BAR>();
      token = sm.token;
      // ---- 7. optional: write the distribution drawn from ------------------------------
      if (G_out) {
        const float invZ = (float)(1.0 / Z);
        for (int tile = warp; tile < ntiles; tile += NT / 32) {
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC];
          rt.load_tile(x0, V, a.vec_ok, zt);
          if (ctx.mode == 0) rd.load_tile(x0, V, a.vec_ok, zd);
#pragma unroll
          for (int k = 0; k < VEC; ++k)
            if (x0 + k < V)
              G_out[x0 + k] = weight_of(rt.filter(zt[k]), ctx.mode == 0 ? rd.filter(zd[k]) : 0.0f, ctx) * invZ;
        }
      }
      break;
    }
  }
  if (G_out && token < 0)
    for (int x = tid; x < V; x += NT) G_out[x] = 0.0f;

  // ---- 8. emit x_{1:tau+1} ---------------------------------------------------------
  if (tid <= L) {
    int v = -1;
    if (tid < tau) v = a.tokens[(int64_t)b * L + tid];
    else if (tid == tau) v = token;
    a.out_tokens[(int64_t)b * (L + 1) + tid] = v;
  }
  if (tid == 0) {
    a.out_accept_len[b] = tau;
    if (a.out_status) a.out_status[b] = status;
  }
  group_sync<NT, BAR>();  // the shared state may be reused for the next sequence
}

template <typename T, bool CFG>
__global__ void __launch_bounds__(kFinishThreads, 1) finish_kernel(const FinishArgs a) {
  extern __shared__ double tile_sums[];  // one fp64 sum per tile
  __shared__ FinishSmem sm;
  pdl_wait();  // everything the statistics kernel wrote is visible from here on
  finish_sequence<T, CFG, kFinishThreads, 0>(a, blockIdx.x, threadIdx.x, tile_sums, sm, 0);
}


// ============================ fused single-launch path ==============================
// One persistent kernel per call.  Phase 1 streams this block's share of the rows
// through a ring of shared-memory stages filled by bulk asynchronous copies
// (the warp that is last to finish reading a stage issues the copy that refills
// it, so nobody waits to produce) and keeps the per-item results in shared memory; nothing is written to global memory yet, so
// phase 1 may overlap the previous call on the stream (programmatic dependent
// launch).  After griddepcontrol.wait, phase 2 publishes the results, counts
// arrivals per sequence, and the block that completes a sequence runs its finish
// -- no block ever waits for another.
//
// Plain mode: an item is one stage-sized chunk of a row.  Top-k mode: an item is a
// whole row, held in registers (64 values per thread, V <= 16384) while its
// threshold is found: a mean/deviation guess `lo` of a value a little below the
// k-th largest, the values >= lo gathered in shared memory, one histogram over
// [lo, max] to find the bin of the k-th largest, an exact rank among that bin's
// few values.  Whenever the guess does not bracket the answer (fewer than k
// values, too many, a crowded bin) the row takes the exact radix select over its
// registers instead, so the result never depends on the guess.
constexpr int kFusedConsumers = 256;
constexpr int kFusedThreads = kFusedConsumers;
constexpr int kStages = 4;
constexpr int kStageBytes = 16384;
constexpr int kStashItems = 1024;
constexpr int kWarpList = 256;                // per-warp capacity of the list of values >= lo
constexpr int kListCap = 8 * kWarpList;
constexpr int kLinBins = 512;
constexpr int kCandCap = 64;
constexpr int kRowRegs = 64;                  // top-k mode: values of the row per thread
constexpr int kTopkMaxV = kRowRegs * kFusedConsumers;
constexpr long long kWaitCycles = 1ll << 31;  // about a second: then give up and flag it

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
// global -> shared bulk copy of `bytes` (multiple of 16; both addresses 16-byte aligned),
// completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}
__device__ __forceinline__ void consumer_sync() { group_sync<kFusedConsumers, 1>(); }
// maximum that returns NaN when either operand is NaN (fmaxf would drop it)
__device__ __forceinline__ float max_nan(float x, float y) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y));
  return r;
}
// bin of v in the linear histogram over [lo, max]; the same instructions wherever it is evaluated
__device__ __forceinline__ int lin_bin(float v, float lo, float scale) {
  return min(kLinBins - 1, (int)__fmul_rn(__fsub_rn(v, lo), scale));
}

struct FusedArgs {
  FinishArgs fin;       // inputs, outputs, partials, thresholds (parts = chunks per row, or 1 with top-k)
  int n_items;          // plain: rows * parts_per_row; top-k: rows
  int chunks_per_row;   // top-k kernel: block stages per row
  int chunks_per_part;  // plain kernel: warp stages per part
  int parts_per_row;    // plain kernel
  int items_per_seq;
  int top_k;
  float lo_sigmas;      // top-k guess: lo = mean + lo_sigmas * deviation (NaN: always take the exact select)
  float* tok_logit;     // [rows] (mixed, unfiltered) logit of the row's drafted token, written in phase 2
  int* counters;        // [B] arrivals per sequence; zero before the first call, left zero by every call
  int* error_flag;      // set when a bounded wait gave up
};

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

// ---- finish with everything staged in shared memory ---------------------------------
// The fused kernels' finish: few dependent round trips to global memory.  One round
// brings the sequence's partials, thresholds, drafted tokens with their logits (found
// in phase 1 while the rows streamed by), uniforms and multipliers into shared
// memory; after the accept tests, bulk copies bring the two rows of position tau+1
// into the 64 KB ring, a segment at a time, and Eq. opt_G is summed from there.
constexpr int kRingBytes = 65536;
constexpr int kFinTiles = 1024;   // tiles of 32 lanes x 16 bytes: V <= 131072 (fp32) / 262144 (bf16)

struct FinishStage {
  int tok[kMaxGamma + 1];
  float uni[kMaxGamma + 1];
  float omega[kMaxGamma];
  float tokz[2 * kMaxGamma + 1];
  float thr_row[2 * kMaxGamma + 1];
  double tile_sums[kFinTiles];
  alignas(8) uint64_t bar;
};

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

template <typename T, bool CFG, int NT, int BAR>
__device__ void finish_sequence_staged(const FusedArgs& ua, const int b, const int tid, unsigned char* ring,
                                       FinishSmem& sm, FinishStage& st, uint32_t& phase, const int extra_status) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int TILE = 32 * VEC;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int ES = (int)sizeof(T);
  const FinishArgs& a = ua.fin;
  const int lane = tid & 31, warp = tid >> 5;
  const int L = a.gamma, V = a.V;
  const int rows_per_seq = a.T + L;
  const T* tgt = reinterpret_cast<const T*>(a.target) + (int64_t)b * a.tstride;
  const T* dft = reinterpret_cast<const T*>(a.draft) + (int64_t)b * a.dstride;
  const T* tgt_u = CFG ? reinterpret_cast<const T*>(a.target_uncond) + (int64_t)b * a.tstride : nullptr;
  const T* dft_u = CFG ? reinterpret_cast<const T*>(a.draft_uncond) + (int64_t)b * a.dstride : nullptr;

  // ---- 0. one round trip: everything the accept tests need ----------------------------
  const int n_entries = rows_per_seq * a.parts;
  float2* staged = reinterpret_cast<float2*>(ring);
  {
    const float2* src = a.partials + (int64_t)b * n_entries;
    for (int idx = tid; idx < n_entries; idx += NT) staged[idx] = __ldcg(src + idx);
    if (tid < L) {
      st.tok[tid] = a.tokens[(int64_t)b * L + tid];
      const float om = a.schedule[tid];
      st.omega[tid] = om >= 0.0f ? om : 0.0f;
    }
    if (tid <= L) st.uni[tid] = a.uniforms[(int64_t)b * (L + 1) + tid];
    if (tid < rows_per_seq) {
      st.thr_row[tid] = a.use_topk ? __ldcg(a.thresholds + (int64_t)b * rows_per_seq + tid) : CSD_NEG_INF;
      st.tokz[tid] = __ldcg(ua.tok_logit + (int64_t)b * rows_per_seq + tid);
    }
  }
  group_sync<NT, BAR>();

  // ---- 1. per position: merge parts, Eq. relax, accept test ------------------------------
  for (int i = warp; i <= L; i += NT / 32) {
    const bool has_t = i < a.T, has_d = i < L;
    float M[2] = {CSD_NEG_INF, CSD_NEG_INF}, S[2] = {-1.0f, -1.0f};
    float thr[2] = {CSD_NEG_INF, CSD_NEG_INF};
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      if (which == 0 ? !has_t : !has_d) continue;
      const int row_local = which == 0 ? i : a.T + i;
      float m = CSD_NEG_INF, s = -1.0f;
      for (int p = lane; p < a.parts; p += 32) {
        const float2 v = staged[row_local * a.parts + p];
        stat_merge(m, s, v.x, v.y);
      }
      stat_warp_allreduce(m, s);
      M[which] = m; S[which] = s;
      thr[which] = st.thr_row[row_local];
    }
    if (lane == 0) {
      const bool t_ok = has_t && M[0] > CSD_NEG_INF && M[0] < CSD_POS_INF && S[0] >= 0.0f && S[0] < CSD_POS_INF;
      const bool d_ok = has_d && M[1] > CSD_NEG_INF && M[1] < CSD_POS_INF && S[1] >= 0.0f && S[1] < CSD_POS_INF;
      sm.M[0][i] = M[0]; sm.S[0][i] = S[0]; sm.thr[0][i] = thr[0];
      sm.M[1][i] = M[1]; sm.S[1][i] = S[1]; sm.thr[1][i] = thr[1];
      sm.valid[0][i] = t_ok; sm.valid[1][i] = d_ok;
      int flag = 0;
      if (i < L) {
        const int tok = st.tok[i];
        const bool tok_ok = tok >= 0 && tok < V;
        const float omega = st.omega[i];
        float f = 0.0f, p = __int_as_float(0x7fc00000), q = p;
        if (!t_ok || !d_ok) flag = 1;
        else if (!tok_ok) flag = 2;
        else {
          const float zt = st.tokz[i], zd = st.tokz[a.T + i];
          const float dt = (zt < thr[0] ? CSD_NEG_INF : zt) - M[0];
          const float dd = (zd < thr[1] ? CSD_NEG_INF : zd) - M[1];
          p = ex2f(dt * kLog2e) / (1.0f + S[0]);
          q = ex2f(dd * kLog2e) / (1.0f + S[1]);
          if (dd == CSD_NEG_INF) f = 1.0f;         // q = 0: p/q = +inf, and 0/0 := 1
          else if (dt == CSD_NEG_INF) f = 0.0f;    // p = 0 < q
          else f = fminf(1.0f, omega * ex2f((dt - dd) * kLog2e) * ((1.0f + S[1]) / (1.0f + S[0])));
        }
        sm.acc[i] = (st.uni[i] <= f) ? 1 : 0;
        if (a.dbg_p) a.dbg_p[(int64_t)b * L + i] = p;
        if (a.dbg_q) a.dbg_q[(int64_t)b * L + i] = q;
        if (a.dbg_f) a.dbg_f[(int64_t)b * L + i] = f;
      }
      sm.flag[i] = flag;
    }
  }
  group_sync<NT, BAR>();

  // ---- 2. tau = number of leading accepts (the for/break of Algorithm 1) --------
  int tau = 0;
  while (tau < L && sm.acc[tau]) ++tau;
  int status = extra_status;
  for (int i = 0; i <= min(tau, L - 1); ++i) status |= sm.flag[i];

  // ---- 3. which row to draw from -------------------------------------------------
  const int j = tau;  // 0-based row index of position tau+1 (j == L: bonus row)
  PairCtx ctx;
  bool draw = true;
  if (j < L) {
    if (!sm.valid[0][j]) draw = false;
    ctx.mode = sm.valid[1][j] ? 0 : 1;
  } else {
    if (a.T == L + 1) {
      ctx.mode = 1;
      if (!sm.valid[0][L]) { draw = false; status |= 1; }
    } else draw = false;
  }
  float* G_out = a.dbg_G ? a.dbg_G + (int64_t)b * V : nullptr;
  const int ntiles = (V + TILE - 1) / TILE;
  int token = -1;

  if (draw) {
    ctx.Mt = sm.M[0][j]; ctx.St = sm.S[0][j];
    ctx.Md = j < L ? sm.M[1][j] : 0.0f; ctx.Sd = j < L ? sm.S[1][j] : 0.0f;
    ctx.inv_t = 1.0f / (1.0f + ctx.St);
    ctx.inv_den = ctx.inv_t / (1.0f + ctx.Sd);
    ctx.one_minus_omega = 1.0f - (j < L ? st.omega[j] : 0.0f);
    Row<T, CFG> rt{tgt + (int64_t)j * V, CFG ? tgt_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[0][j]};
    Row<T, CFG> rd = rt;
    if (j < L) rd = Row<T, CFG>{dft + (int64_t)j * V, CFG ? dft_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[1][j]};
    const float u = st.uni[L];

    for (int attempt = 0; attempt < 2; ++attempt) {
      // ---- 4. Eq. opt_G weights: the rows come through the ring, one fp64 sum per tile ------
      const int n_arr = (ctx.mode == 0 ? 2 : 1) * ARR;
      const int seg_elems = (kRingBytes / n_arr / (TILE * ES)) * TILE;   // elements of each array per segment
      const int slot_bytes = seg_elems * ES;
      for (int x0 = 0; x0 < V; x0 += seg_elems) {
        group_sync<NT, BAR>();   // everybody is done with what the ring held
        const int n = min(seg_elems, V - x0);
        if (tid == 0) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          const uint32_t bytes = (uint32_t)(n * ES);
          mbar_expect_tx(&st.bar, bytes * n_arr);
          bulk_load(ring, rt.cond + x0, bytes, &st.bar);
          if (CFG) bulk_load(ring + slot_bytes, rt.uncond + x0, bytes, &st.bar);
          if (ctx.mode == 0) {
            bulk_load(ring + ARR * slot_bytes, rd.cond + x0, bytes, &st.bar);
            if (CFG) bulk_load(ring + (ARR + 1) * slot_bytes, rd.uncond + x0, bytes, &st.bar);
          }
        }
        if (!mbar_wait(&st.bar, phase)) status |= 8;
        phase ^= 1u;
        const int seg_tiles = (n + TILE - 1) / TILE;
        for (int t = warp; t < seg_tiles; t += NT / 32) {
          const int xo = t * TILE + lane * VEC;   // offset inside the segment
          float acc = 0.0f;
          if (xo < n) {
            float zt[VEC], zd[VEC];
            unpack_vec<T>(ring + xo * ES, zt);
            if (CFG) {
              float zu[VEC];
              unpack_vec<T>(ring + slot_bytes + xo * ES, zu);
#pragma unroll
              for (int k = 0; k < VEC; ++k) zt[k] = cfg_mix(zt[k], zu[k], a.cfg_scale);
            }
            if (ctx.mode == 0) {
              unpack_vec<T>(ring + ARR * slot_bytes + xo * ES, zd);
              if (CFG) {
                float zu[VEC];
                unpack_vec<T>(ring + (ARR + 1) * slot_bytes + xo * ES, zu);
#pragma unroll
                for (int k = 0; k < VEC; ++k) zd[k] = cfg_mix(zd[k], zu[k], a.cfg_scale);
              }
            }
#pragma unroll
            for (int k = 0; k < VEC; ++k)
              acc += weight_of(rt.filter(zt[k]), ctx.mode == 0 ? rd.filter(zd[k]) : 0.0f, ctx);
          }
          const double tsum = warp_sum_double((double)acc);
          if (lane == 0) st.tile_sums[x0 / TILE + t] = tsum;
        }
      }
      group_sync<NT, BAR>();
      // ---- 5. locate the tile that holds the crossing C(x) > u Z ------------------
      if (warp == 0) {
        const int chunk = (ntiles + 31) / 32;
        const int t0 = lane * chunk, t1 = min(ntiles, t0 + chunk);
        double local = 0.0;
        for (int t = t0; t < t1; ++t) local += st.tile_sums[t];
        const double incl = warp_incl_scan_double(local, lane);
        const double Z = __shfl_sync(0xffffffffu, incl, 31);
        const double target = (double)u * Z;
        const bool mine = incl > target && local > 0.0;
        const unsigned ballot = __ballot_sync(0xffffffffu, mine);
        if (lane == 0) { sm.Z = Z; sm.pick_tile = -1; }
        __syncwarp();
        if (ballot != 0 && lane == __ffs(ballot) - 1) {
          double c = incl - local, c_pick = c;
          int pick = t0;
          for (int t = t0; t < t1; ++t) {
            const double v = st.tile_sums[t];
            if (v > 0.0) { pick = t; c_pick = c; }   // last tile with mass seen so far
            if (c + v > target && v > 0.0) break;
            c += v;
          }
          sm.pick_tile = pick;
          sm.pick_prefix = c_pick;
        }
      }
      group_sync<NT, BAR>();
      const double Z = sm.Z;
      if (!(Z > 0.0) || !(Z < (double)CSD_POS_INF)) {
        if (attempt == 0 && ctx.mode == 0) {  // empty positive part: fall back to G := P_j
          ctx.mode = 1;
          status |= 4;
          continue;
        }
        break;  // nothing to draw from
      }
      // ---- 6. scan inside that tile (its 32 vectors come from global memory again) -----------
      if (warp == 0) {
        const int tile = sm.pick_tile;
        const double target = (double)u * Z;
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC], zd[VEC];
        rt.load_tile(x0, V, 1, zt);
        if (ctx.mode == 0) rd.load_tile(x0, V, 1, zd);
        double run[VEC];
        double acc = 0.0;
        int last_pos = -1;
        unsigned posmask = 0;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          const float g = weight_of(rt.filter(zt[k]), ctx.mode == 0 ? rd.filter(zd[k]) : 0.0f, ctx);
          if (g > 0.0f) { last_pos = k; posmask |= 1u << k; }
          acc += (double)g;
          run[k] = acc;
        }
        const double before = sm.pick_prefix + (warp_incl_scan_double(acc, lane) - acc);
        int first = -1;
#pragma unroll
        for (int k = VEC - 1; k >= 0; --k)
          if (before + run[k] > target && ((posmask >> k) & 1u)) first = k;
        const unsigned hit = __ballot_sync(0xffffffffu, first >= 0);
        const unsigned pos = __ballot_sync(0xffffffffu, last_pos >= 0);
        if (hit != 0) {
          if (lane == __ffs(hit) - 1) sm.token = x0 + first;
        } else if (pos != 0) {  // rounding left no crossing: last token with positive weight
          if (lane == 31 - __clz(pos)) sm.token = x0 + last_pos;
        } else if (lane == 0) sm.token = -1;
      }
      group_sync<NT, BAR>();
      token = sm.token;
      // ---- 7. optional: write the distribution drawn from ------------------------------
      if (G_out) {
        const float invZ = (float)(1.0 / Z);
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
      break;
    }
  }
  if (G_out && token < 0)
    for (int x = tid; x < V; x += NT) G_out[x] = 0.0f;

  // ---- 8. emit x_{1:tau+1} ---------------------------------------------------------
  if (tid <= L) {
    int v = -1;
    if (tid < tau) v = st.tok[tid];
    else if (tid == tau) v = token;
    a.out_tokens[(int64_t)b * (L + 1) + tid] = v;
  }
  if (tid == 0) {
    a.out_accept_len[b] = tau;
    if (a.out_status) a.out_status[b] = status;
  }
  group_sync<NT, BAR>();  // the shared state may be reused for the next sequence
}

struct SelectSmem {
  alignas(16) int hist[kSelectBins];  // linear histogram (first kLinBins bins); all bins in the radix select
  float list[8][kWarpList];         // per warp: its values >= lo
  float cand[kCandCap];             // values in the bin of the k-th largest
  float mom[8][4];                  // per warp: sum, sum of squares, count of the sampled values
  float wmax[8];
  int wcount[8];                    // per warp: length of its list, -1 if it overflowed
  int n_cand[2];                    // by row parity
  float part_acc[2][8];             // per warp, by row parity: sum of exp(z - max) over kept non-maximum values
  int part_cmax[2][8];              //                          number of kept values equal to the maximum
  float part_max[2];
  float part_thr[2];
  int bc_i[4];
  float red_f[8][2];
};

struct FusedSmem {
  alignas(128) unsigned char ring[kStages][kStageBytes];
  alignas(8) uint64_t full[kStages];
  int readers_done[kStages];   // warps that have finished reading the stage's current contents
  float2 stash[kStashItems];
  float stash_thr[kStashItems];
  float stash_tokz[kStashItems];   // logit of the row's drafted token
  int done[kStashItems];
  int n_done;
  int abort;
  FinishSmem fin;
  FinishStage fst;
  SelectSmem sel;
};

// Exact k-th largest of the block's register-resident values (radix select, 11+11+10 bits).
template <int N>
__device__ float radix_select_registers(const float (&z)[N], int k, SelectSmem& ss, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0, mask = 0;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nbins = pass == 2 ? 1024 : 2048;
    for (int d = tid; d < nbins; d += kFusedConsumers) ss.hist[d] = 0;
    consumer_sync();
#pragma unroll
    for (int e = 0; e < N; ++e) {
      const uint32_t key = order_key(z[e]);
      if ((key & mask) == prefix) atomicAdd(&ss.hist[(key >> shift) & (nbins - 1)], 1);
    }
    consumer_sync();
    if (warp == 0) {
      int above;
      const int bin = select_bin_from_top(ss.hist, nbins, k, lane, &above);
      if (lane == 0) { ss.bc_i[0] = (int)(prefix | ((uint32_t)bin << shift)); ss.bc_i[1] = k - above; }
    }
    consumer_sync();
    prefix = (uint32_t)ss.bc_i[0];
    k = ss.bc_i[1];
    mask |= (uint32_t)(nbins - 1) << shift;
    consumer_sync();
  }
  return order_value(prefix);
}

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

template <typename T, bool CFG>
__global__ void __launch_bounds__(kFusedThreads, 2) verify_topk_kernel(const FusedArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int EPS = kStageBytes / ((int)sizeof(T) * ARR);   // elements of a row per stage
  constexpr int VPT = EPS / kFusedConsumers;                  // values per thread per stage
  constexpr int NVS = VPT / VEC;                              // 16-byte vectors per thread per stage
  constexpr int MAXC = kRowRegs / VPT;                        // stages a row may span
  extern __shared__ __align__(128) unsigned char fused_smem_raw[];
  FusedSmem& sm = *reinterpret_cast<FusedSmem*>(fused_smem_raw);
  SelectSmem& ss = sm.sel;

  pdl_launch_dependents();  // the next call on the stream may start its own phase 1

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const FinishArgs& f = a.fin;
  const int V = f.V;
  const int rows_per_seq = f.T + f.gamma;
  const int cpi = a.chunks_per_row;   // stages per row
  const int k_top = a.top_k;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); sm.readers_done[s] = 0; }
    mbar_init(&sm.fst.bar, 1);
    sm.n_done = 0;
    sm.abort = 0;
    sm.sel.n_cand[0] = 0;
    sm.sel.n_cand[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // this block's rows: a contiguous range, so that a sequence's rows sit in few blocks and
  // the finishes spread over the grid
  const int item_begin = (int)((long long)a.n_items * blockIdx.x / gridDim.x);
  const int item_end = (int)((long long)a.n_items * (blockIdx.x + 1) / gridDim.x);

  auto row_pointers = [&](int row_id, const T*& cond, const T*& uncond) {
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    if (r < f.T) {
      const int64_t off = (int64_t)b * f.tstride + (int64_t)r * V;
      cond = reinterpret_cast<const T*>(f.target) + off;
      uncond = CFG ? reinterpret_cast<const T*>(f.target_uncond) + off : nullptr;
    } else {
      const int64_t off = (int64_t)b * f.dstride + (int64_t)(r - f.T) * V;
      cond = reinterpret_cast<const T*>(f.draft) + off;
      uncond = CFG ? reinterpret_cast<const T*>(f.draft_uncond) + off : nullptr;
    }
  };
  auto token_of_row = [&](int row_id) -> int {
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    const int i = r < f.T ? r : r - f.T;
    return i < f.gamma ? __ldg(f.tokens + (int64_t)b * f.gamma + i) : -1;
  };
  // Issues the copies of this block's q-th chunk (if there is one) into stage q % kStages.
  auto issue_chunk = [&](int q) {
    const int j = q / cpi;
    const int c = q - j * cpi;
    const int row_id = item_begin + j;
    if (row_id >= item_end) return;
    const T *cond, *uncond;
    row_pointers(row_id, cond, uncond);
    const int s = q % kStages;
    const int x0 = c * EPS;
    const uint32_t bytes = (uint32_t)(min(EPS, V - x0) * (int)sizeof(T));
    mbar_expect_tx(&sm.full[s], bytes * ARR);
    bulk_load(&sm.ring[s][0], cond + x0, bytes, &sm.full[s]);
    if (CFG) bulk_load(&sm.ring[s][kStageBytes / 2], uncond + x0, bytes, &sm.full[s]);
  };
  if (tid == 0) {
    for (int q = 0; q < kStages; ++q) issue_chunk(q);
  }

  // Merges the eight per-warp partials of a finished row (parity par) into its stash entry.
  auto stash_row = [&](int idx, int par) {
    float tot = 0.0f;
    int ctot = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { tot += ss.part_acc[par][w]; ctot += ss.part_cmax[par][w]; }
    if (idx < kStashItems) {
      sm.stash[idx] = make_float2(ss.part_max[par], tot + (float)(ctot - 1));
      sm.stash_thr[idx] = ss.part_thr[par];
    }
  };

  // ================================= phase 1 ===========================================
  int n_my = 0;
  {
    int q = 0;
    bool ok = true;
    int tok_next = item_begin < item_end ? token_of_row(item_begin) : -1;
    for (int row_id = item_begin; row_id < item_end; ++row_id, ++n_my) {
      const int par = n_my & 1;
      const int tok_cur = tok_next;
      if (row_id + 1 < item_end) tok_next = token_of_row(row_id + 1);
      float zrow[kRowRegs];
#pragma unroll
      for (int e = 0; e < kRowRegs; ++e) zrow[e] = CSD_NEG_INF;
      float mx4[4] = {CSD_NEG_INF, CSD_NEG_INF, CSD_NEG_INF, CSD_NEG_INF};
      float sum1 = 0.0f, sum2 = 0.0f, n_sample = 0.0f;
#pragma unroll
      for (int c = 0; c < MAXC; ++c) {
        if (c < cpi) {
          const int s = q % kStages, round = q / kStages;
          ++q;
          if (ok && !mbar_wait(&sm.full[s], round & 1)) ok = false;
          const int x0 = c * EPS;
          const int n = min(EPS, V - x0);
#pragma unroll
          for (int v = 0; v < NVS; ++v) {
            const int xo = (v * kFusedConsumers + tid) * VEC;
            float zc[VEC];
            if (ok && xo < n) {
              unpack_vec<T>(&sm.ring[s][xo * (int)sizeof(T)], zc);
              if (CFG) {
                float zu[VEC];
                unpack_vec<T>(&sm.ring[s][kStageBytes / 2 + xo * (int)sizeof(T)], zu);
#pragma unroll
                for (int e = 0; e < VEC; ++e) zc[e] = cfg_mix(zc[e], zu[e], f.cfg_scale);
              }
              if (c == 0) {   // the first stage is the sample for the threshold guess
#pragma unroll
                for (int e = 0; e < VEC; ++e) { sum1 += zc[e]; sum2 = fmaf(zc[e], zc[e], sum2); }
                n_sample += (float)VEC;
              }
            } else {
#pragma unroll
              for (int e = 0; e < VEC; ++e) zc[e] = ok ? CSD_NEG_INF : __int_as_float(0x7fc00000);
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              zrow[c * VPT + v * VEC + e] = zc[e];
              mx4[e & 3] = max_nan(mx4[e & 3], zc[e]);
            }
          }
          const int tl = tok_cur - x0;
          if (tid == 0 && ok && tl >= 0 && tl < n) {   // the drafted token's logit passes by: keep it
            float zc = load_scalar_smem<T>(&sm.ring[s][tl * (int)sizeof(T)]);
            if (CFG) zc = cfg_mix(zc, load_scalar_smem<T>(&sm.ring[s][kStageBytes / 2 + tl * (int)sizeof(T)]), f.cfg_scale);
            if (n_my < kStashItems) sm.stash_tokz[n_my] = zc;
          }
          __syncwarp();
          if (lane == 0) {   // this warp is done with the stage; the last one to say so refills it
            __threadfence_block();
            if (atomicAdd(&sm.readers_done[s], 1) == kFusedConsumers / 32 - 1) {
              sm.readers_done[s] = 0;
              __threadfence_block();
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              issue_chunk(q - 1 + kStages);
            }
          }
          if (c == 0) {   // publish the sample's moments early: the reduction overlaps the other stages
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
              sum1 += __shfl_xor_sync(0xffffffffu, sum1, off);
              sum2 += __shfl_xor_sync(0xffffffffu, sum2, off);
              n_sample += __shfl_xor_sync(0xffffffffu, n_sample, off);
            }
            if (lane == 0) { ss.mom[warp][0] = sum1; ss.mom[warp][1] = sum2; ss.mom[warp][2] = n_sample; }
          }
        }
      }
      float mx = max_nan(max_nan(mx4[0], mx4[1]), max_nan(mx4[2], mx4[3]));
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = max_nan(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      if (lane == 0) ss.wmax[warp] = mx;
      for (int d = tid; d < kLinBins; d += kFusedConsumers) ss.hist[d] = 0;
      consumer_sync();   // ---- A: moments, maxima, cleared histogram; the previous row's partials are complete
      if (tid == 0) {
        ss.n_cand[par ^ 1] = 0;   // for the next row; nobody reads the previous row's count any more
        if (n_my > 0) stash_row(n_my - 1, par ^ 1);
      }
      float s1 = 0.0f, s2 = 0.0f, nn = 0.0f;
      mx = ss.wmax[0];
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        s1 += ss.mom[w][0]; s2 += ss.mom[w][1]; nn += ss.mom[w][2];
        mx = max_nan(mx, ss.wmax[w]);
      }
      const float mean = s1 / nn;
      const float lo = mean + a.lo_sigmas * sqrtf(fmaxf(s2 / nn - mean * mean, 0.0f));
      const float scale = (float)kLinBins / (mx - lo);
      // ---- this warp's values >= lo: into its list and into the histogram ----------------
      int cnt = 0;
#pragma unroll
      for (int e = 0; e < kRowRegs; ++e) cnt += (zrow[e] >= lo) ? 1 : 0;
      int incl = cnt;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
      }
      const int wc = __shfl_sync(0xffffffffu, incl, 31);
      const bool usable = (mx > lo) && (mx < CSD_POS_INF);   // false for NaN guesses and NaN / +inf rows
      if (wc <= kWarpList && usable) {
        int pos = incl - cnt;
#pragma unroll
        for (int e = 0; e < kRowRegs; ++e) {
          if (zrow[e] >= lo) {
            ss.list[warp][pos++] = zrow[e];
            atomicAdd(&ss.hist[lin_bin(zrow[e], lo, scale)], 1);
          }
        }
      }
      if (lane == 0) ss.wcount[warp] = (wc <= kWarpList && usable) ? wc : -1;
      consumer_sync();   // ---- B: lists and histogram complete
      int n_lo = 0;
      bool fast = true;
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const int c = ss.wcount[w];
        if (c < 0) fast = false;
        n_lo += c;
      }
      fast = fast && n_lo >= k_top;
      float thr = CSD_NEG_INF;
      if (fast) {
        int kk;
        const int pick_bin = warp_pick_bin(ss.hist, k_top, lane, &kk);   // every warp computes it for itself
        for (int i = lane; i < wc; i += 32) {
          const float v = ss.list[warp][i];
          if (lin_bin(v, lo, scale) == pick_bin) {
            const int slot = atomicAdd(&ss.n_cand[par], 1);
            if (slot < kCandCap) ss.cand[slot] = v;
          }
        }
        consumer_sync();   // ---- D: candidates complete
        const int n_cand = ss.n_cand[par];
        if (n_cand <= kCandCap) {
          // exact rank among the candidates, every warp for itself (two candidates per lane)
          const float v0 = lane < n_cand ? ss.cand[lane] : CSD_NEG_INF;
          const float v1 = lane + 32 < n_cand ? ss.cand[lane + 32] : CSD_NEG_INF;
          int gt0 = 0, ge0 = 0, gt1 = 0, ge1 = 0;
          for (int j2 = 0; j2 < n_cand; ++j2) {
            const float w = ss.cand[j2];
            gt0 += (w > v0) ? 1 : 0; ge0 += (w >= v0) ? 1 : 0;
            gt1 += (w > v1) ? 1 : 0; ge1 += (w >= v1) ? 1 : 0;
          }
          const bool hit0 = lane < n_cand && gt0 < kk && kk <= ge0;
          const bool hit1 = lane + 32 < n_cand && gt1 < kk && kk <= ge1;
          const unsigned b0 = __ballot_sync(0xffffffffu, hit0);
          const unsigned b1 = __ballot_sync(0xffffffffu, hit1);
          thr = b0 ? __shfl_sync(0xffffffffu, v0, __ffs(b0) - 1) : __shfl_sync(0xffffffffu, v1, b1 ? __ffs(b1) - 1 : 0);
          // ---- statistics of the kept values of this warp's list -------------------------
          float acc = 0.0f;
          int cmax = 0;
          for (int i = lane; i < wc; i += 32) {
            const float v = ss.list[warp][i];
            if (v >= thr) {
              if (v == mx) cmax += 1;
              else acc += ex2f((v - mx) * kLog2e);
            }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            acc += __shfl_xor_sync(0xffffffffu, acc, off);
            cmax += __shfl_xor_sync(0xffffffffu, cmax, off);
          }
          if (lane == 0) { ss.part_acc[par][warp] = acc; ss.part_cmax[par][warp] = cmax; }
          if (tid == 0) { ss.part_max[par] = mx; ss.part_thr[par] = thr; }
          continue;   // the partials are merged after the next barrier
        }
        fast = false;   // crowded bin (the same decision in every thread: n_cand is shared)
      }
      // ---- exact select over the registers, statistics from the registers ---------------
      consumer_sync();
      thr = radix_select_registers(zrow, k_top, ss, tid);
      float m = CSD_NEG_INF;
#pragma unroll
      for (int e = 0; e < kRowRegs; ++e) m = fmaxf(m, zrow[e]);   // the maximum always passes the filter (k >= 1)
      float acc = 0.0f;
      int cnt2 = 0;
#pragma unroll
      for (int e = 0; e < kRowRegs; ++e) {
        const float v = zrow[e] < thr ? CSD_NEG_INF : zrow[e];
        const float ex = ex2f((v - m) * kLog2e);
        if (v == m) cnt2 += 1; else acc += ex;          // NaN entries poison acc, which marks the row
      }
      float s_loc = acc + (float)(cnt2 - 1);
      stat_warp_allreduce(m, s_loc);
      if (lane == 0) { ss.red_f[warp][0] = m; ss.red_f[warp][1] = s_loc; }
      consumer_sync();
      if (tid == 0) {
        float mm = ss.red_f[0][0], sv = ss.red_f[0][1];
#pragma unroll
        for (int w = 1; w < 8; ++w) stat_merge(mm, sv, ss.red_f[w][0], ss.red_f[w][1]);
        // same form as the fast path's partials: one "maximum", the rest in warp 0's slot
#pragma unroll
        for (int w = 0; w < 8; ++w) { ss.part_acc[par][w] = 0.0f; ss.part_cmax[par][w] = 0; }
        ss.part_acc[par][0] = sv;
        ss.part_cmax[par][0] = 1;
        ss.part_max[par] = mm;
        ss.part_thr[par] = thr;
      }
    }
    consumer_sync();
    if (tid == 0 && n_my > 0) stash_row(n_my - 1, (n_my - 1) & 1);
    if (!ok && tid == 0) {
      sm.abort = 1;
      atomicExch(a.error_flag, 1);
      // copies issued for stages this thread gave up on may still be in flight: wait for them, again bounded
      for (int s = 0; s < kStages; ++s)
        if (q > s) (void)mbar_wait(&sm.full[s], ((q - 1 - s) / kStages) & 1);
    }
  }

  // ================================= phase 2 ===========================================
  pdl_wait();   // the previous call on the stream has finished with the workspace and the outputs
  consumer_sync();
  for (int idx = tid; idx < n_my; idx += kFusedConsumers) {
    const int row_id = item_begin + idx;
    const_cast<float2*>(f.partials)[row_id] = sm.stash[idx];
    const_cast<float*>(f.thresholds)[row_id] = sm.stash_thr[idx];
    a.tok_logit[row_id] = sm.stash_tokz[idx];
  }
  __threadfence();
  consumer_sync();
  for (int idx = tid; idx < n_my; idx += kFusedConsumers) {
    const int b = (item_begin + idx) / rows_per_seq;
    __threadfence();
    const int old = atomicAdd(&a.counters[b], 1);
    if (old + 1 == a.items_per_seq) {
      const int slot = atomicAdd(&sm.n_done, 1);
      sm.done[slot] = b;
    }
  }
  consumer_sync();
  const int n_done = sm.n_done;
  if (n_done > 0) {
    __threadfence();
    const int extra = (sm.abort || __ldcg(a.error_flag)) ? 8 : 0;
    uint32_t fin_phase = 0;
    for (int d = 0; d < n_done; ++d) {
      const int b = sm.done[d];
      finish_sequence_staged<T, CFG, kFusedConsumers, 1>(a, b, tid, &sm.ring[0][0], sm.fin, sm.fst, fin_phase, extra);
      if (tid == 0) a.counters[b] = 0;   // ready for the next call
    }
  }
}

// ---- plain kernel: every warp streams its own parts through its own ring -----------
// No block-level step in phase 1: a warp owns a contiguous range of items (an item is
// a part of a row: chunks_per_part warp stages), a private ring of kWStages stages
// of kWStageBytes, issues its own refills, and keeps a running (m, s) per lane that it
// reduces once per item.  Eight such pipelines per block sit at different points of their
// loops and hide each other's latencies.
constexpr int kWStages = 4;
constexpr int kWStageBytes = 2048;
constexpr int kWarpStash = 128;
constexpr int kPlainWarps = kFusedConsumers / 32;

struct PlainSmem {
  alignas(128) unsigned char ring[kPlainWarps][kWStages][kWStageBytes];
  alignas(8) uint64_t full[kPlainWarps][kWStages];
  float2 stash[kPlainWarps][kWarpStash];
  float stash_tokz[kPlainWarps][kWarpStash];   // logit of the row's drafted token, if this part holds it
  unsigned char stash_has[kPlainWarps][kWarpStash];
  int done[kPlainWarps * kWarpStash];
  int n_done;
  int abort;
  FinishSmem fin;
  FinishStage fst;
};

template <typename T, bool CFG>
__global__ void __launch_bounds__(kFusedThreads, 2) verify_plain_kernel(const FusedArgs a) {
  constexpr int VEC = Elem<T>::kVec;
  constexpr int ARR = CFG ? 2 : 1;
  constexpr int EPS = kWStageBytes / ((int)sizeof(T) * ARR);   // elements of a row per warp stage
  constexpr int VPL = EPS / 32;                                // values per lane per stage
  constexpr int NVS = VPL / VEC;                               // 16-byte vectors per lane per stage
  extern __shared__ __align__(128) unsigned char fused_smem_raw[];
  PlainSmem& sm = *reinterpret_cast<PlainSmem*>(fused_smem_raw);

  pdl_launch_dependents();  // the next call on the stream may start its own phase 1

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const FinishArgs& f = a.fin;
  const int V = f.V;
  const int rows_per_seq = f.T + f.gamma;
  const int part_elems = a.chunks_per_part * EPS;

  if (tid == 0) { sm.n_done = 0; sm.abort = 0; mbar_init(&sm.fst.bar, 1); }
  if (lane == 0) {
    for (int s = 0; s < kWStages; ++s) mbar_init(&sm.full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const long long gw = (long long)blockIdx.x * kPlainWarps + warp;
  const long long GW = (long long)gridDim.x * kPlainWarps;
  const int item_begin = (int)((long long)a.n_items * gw / GW);
  const int item_end = (int)((long long)a.n_items * (gw + 1) / GW);

  // producer cursor (lane 0): the next chunk to copy
  int p_item = item_begin, p_x = 0, p_xend = 0, p_q = 0;
  const T *p_cond = nullptr, *p_uncond = nullptr;
  auto producer_open_item = [&]() {   // sets the cursor to the first chunk of p_item
    const int row_id = p_item / a.parts_per_row;
    const int part = p_item - row_id * a.parts_per_row;
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    int64_t off;
    if (r < f.T) {
      off = (int64_t)b * f.tstride + (int64_t)r * V;
      p_cond = reinterpret_cast<const T*>(f.target) + off;
      p_uncond = CFG ? reinterpret_cast<const T*>(f.target_uncond) + off : nullptr;
    } else {
      off = (int64_t)b * f.dstride + (int64_t)(r - f.T) * V;
      p_cond = reinterpret_cast<const T*>(f.draft) + off;
      p_uncond = CFG ? reinterpret_cast<const T*>(f.draft_uncond) + off : nullptr;
    }
    p_x = part * part_elems;
    p_xend = min(V, p_x + part_elems);
  };
  auto producer_issue = [&]() {       // copies one chunk into stage p_q % kWStages, if any is left
    if (p_item >= item_end) return;
    const int s = p_q % kWStages;
    const uint32_t bytes = (uint32_t)(min(EPS, p_xend - p_x) * (int)sizeof(T));
    mbar_expect_tx(&sm.full[warp][s], bytes * ARR);
    bulk_load(&sm.ring[warp][s][0], p_cond + p_x, bytes, &sm.full[warp][s]);
    if (CFG) bulk_load(&sm.ring[warp][s][kWStageBytes / 2], p_uncond + p_x, bytes, &sm.full[warp][s]);
    ++p_q;
    p_x += EPS;
    if (p_x >= p_xend) {
      ++p_item;
      if (p_item < item_end) producer_open_item();
    }
  };
  if (lane == 0 && item_begin < item_end) {
    producer_open_item();
    for (int s = 0; s < kWStages; ++s) producer_issue();
  }

  // drafted token of a row (-1 for the bonus row), loaded a row ahead of its use
  auto token_of_row = [&](int row_id) -> int {
    const int b = row_id / rows_per_seq;
    const int r = row_id - b * rows_per_seq;
    const int i = r < f.T ? r : r - f.T;
    return i < f.gamma ? __ldg(f.tokens + (int64_t)b * f.gamma + i) : -1;
  };

  // ================================= phase 1 ===========================================
  int n_my = 0;
  {
    int q = 0;
    bool ok = true;
    int cur_row = -1, tok_cur = -1, tok_next = -1;
    const int last_row = item_end > item_begin ? (item_end - 1) / a.parts_per_row : -1;
    if (item_begin < item_end) tok_next = token_of_row(item_begin / a.parts_per_row);
    for (int item = item_begin; item < item_end; ++item, ++n_my) {
      const int row_id = item / a.parts_per_row;
      const int part = item - row_id * a.parts_per_row;
      const int x_begin = part * part_elems;
      const int x_end = min(V, x_begin + part_elems);
      if (row_id != cur_row) {
        cur_row = row_id;
        tok_cur = tok_next;
        if (row_id < last_row) tok_next = token_of_row(row_id + 1);
      }
      float tokz = 0.0f;
      bool has_tok = false;
      float m = CSD_NEG_INF, s_acc = -1.0f;
      for (int x0 = x_begin; x0 < x_end; x0 += EPS, ++q) {
        const int s = q % kWStages, round = q / kWStages;
        if (ok && !mbar_wait(&sm.full[warp][s], round & 1)) ok = false;
        const int n = min(EPS, x_end - x0);
        float vals[VPL];
#pragma unroll
        for (int v = 0; v < NVS; ++v) {
          const int xo = (v * 32 + lane) * VEC;
          float zc[VEC];
          if (ok && xo < n) {
            unpack_vec<T>(&sm.ring[warp][s][xo * (int)sizeof(T)], zc);
            if (CFG) {
              float zu[VEC];
              unpack_vec<T>(&sm.ring[warp][s][kWStageBytes / 2 + xo * (int)sizeof(T)], zu);
#pragma unroll
              for (int e = 0; e < VEC; ++e) zc[e] = cfg_mix(zc[e], zu[e], f.cfg_scale);
            }
          } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) zc[e] = ok ? CSD_NEG_INF : __int_as_float(0x7fc00000);
          }
#pragma unroll
          for (int e = 0; e < VEC; ++e) vals[v * VEC + e] = zc[e];
        }
        const int tl = tok_cur - x0;
        if (ok && tl >= 0 && tl < n) {   // the drafted token's logit passes by: keep it
          float zc = load_scalar_smem<T>(&sm.ring[warp][s][tl * (int)sizeof(T)]);
          if (CFG) zc = cfg_mix(zc, load_scalar_smem<T>(&sm.ring[warp][s][kWStageBytes / 2 + tl * (int)sizeof(T)]), f.cfg_scale);
          tokz = zc;
          has_tok = true;
        }
        __syncwarp();
        if (lane == 0) {   // the stage is free again: refill it with the chunk kWStages ahead
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          producer_issue();
        }
        float m1, s1;
        stat_of_values(vals, m1, s1);
        if (lane * VEC < n || !ok) stat_merge(m, s_acc, m1, s1);
      }
      stat_warp_allreduce(m, s_acc);
      if (lane == 0 && n_my < kWarpStash) {
        sm.stash[warp][n_my] = make_float2(m, s_acc);
        sm.stash_tokz[warp][n_my] = tokz;
        sm.stash_has[warp][n_my] = has_tok ? 1 : 0;
      }
    }
    if (!ok && lane == 0) {
      sm.abort = 1;
      atomicExch(a.error_flag, 1);
      for (int s = 0; s < kWStages; ++s)   // copies this warp gave up on may still be in flight
        if (q > s) (void)mbar_wait(&sm.full[warp][s], ((q - 1 - s) / kWStages) & 1);
    }
  }

  // ================================= phase 2 ===========================================
  pdl_wait();   // the previous call on the stream has finished with the workspace and the outputs
  __syncwarp();
  for (int idx = lane; idx < n_my; idx += 32) {
    const_cast<float2*>(f.partials)[item_begin + idx] = sm.stash[warp][idx];
    if (sm.stash_has[warp][idx]) a.tok_logit[(item_begin + idx) / a.parts_per_row] = sm.stash_tokz[warp][idx];
  }
  __threadfence();
  __syncthreads();
  for (int idx = lane; idx < n_my; idx += 32) {
    const int row_id = (item_begin + idx) / a.parts_per_row;
    const int b = row_id / rows_per_seq;
    __threadfence();
    const int old = atomicAdd(&a.counters[b], 1);
    if (old + 1 == a.items_per_seq) {
      const int slot = atomicAdd(&sm.n_done, 1);
      sm.done[slot] = b;
    }
  }
  __syncthreads();
  const int n_done = sm.n_done;
  if (n_done > 0) {
    __threadfence();
    const int extra = (sm.abort || __ldcg(a.error_flag)) ? 8 : 0;
    uint32_t fin_phase = 0;
    for (int d = 0; d < n_done; ++d) {
      const int b = sm.done[d];
      finish_sequence_staged<T, CFG, kFusedThreads, 0>(a, b, tid, &sm.ring[0][0][0], sm.fin, sm.fst, fin_phase, extra);
      if (tid == 0) a.counters[b] = 0;   // ready for the next call
    }
  }
}

}  // namespace csd
