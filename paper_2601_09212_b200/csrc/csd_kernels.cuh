// Device code of libcsd: the verify-and-resample round of Cool-SD on sm_100a.
// This file holds the shared arithmetic and the multi-launch path used for rows that
// are unaligned or tiny; the single-launch path that normal calls take is in
// csd_fused.cuh.
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

// Shared-memory atomic add issued as written (the compiler's warp-aggregated form of atomicAdd costs
// about ten instructions; these are called by one lane per warp)
__device__ __forceinline__ int atom_add_shared(int* p, int v) {
  int old;
  asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- (m, s) algebra ---------------------------------------------------------
// identity: m = -inf, s = -1 (so that 1 + s = 0)
__device__ __forceinline__ void stat_merge(float& m, float& s, float m2, float s2) {
  if (m2 > m) {
    float t = m; m = m2; m2 = t;
    t = s; s = s2; s2 = t;
  }
  if (m2 != CSD_NEG_INF) s += (1.0f + s2) * ex2f((m2 - m) * kLog2e);
  else s += s2 - s2;   // nothing to add, but a NaN sum (a NaN beside nothing but masked values) must survive
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

// ---- checked build ------------------------------------------------------------
// With -DCSD_CHECKED every element access of a logit row whose index comes from the data (a drafted
// token, a neighbour id) or from the row length is tested against the row's length first; a bad
// index is recorded (count, first index, the length it was tested against, a site tag) and the access
// is skipped (it reads -inf), so nothing can fault.  The normal build has none of this.
__device__ int g_checked[4];
#ifdef CSD_CHECKED
#define CSD_ROW_LEN(len) , (len)
__device__ __forceinline__ bool checked_ok(int idx, int width, int n, int site) {
  if (idx >= 0 && idx + width <= n) return true;
  if (atomicAdd(&g_checked[0], 1) == 0) { g_checked[1] = idx; g_checked[2] = n; g_checked[3] = site; }
  return false;
}
#else
#define CSD_ROW_LEN(len)
#endif

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

// ---- two fp32 operations per instruction (packed fp32 pairs in 64-bit registers) -----------------
// Each half is the IEEE operation, so results are bit-identical to the scalar forms.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// cfg_mix of VEC values in pairs: c - u as fma(u, -1, c) (one rounding, like the subtraction)
template <int VEC>
__device__ __forceinline__ void cfg_mix_vec(float (&c)[VEC], const float (&u)[VEC], float s) {
  const uint64_t s2 = pack2(s, s), m1 = pack2(-1.0f, -1.0f);
#pragma unroll
  for (int k = 0; k < VEC; k += 2) {
    const uint64_t u2 = pack2(u[k], u[k + 1]);
    const uint64_t d2 = fma2(u2, m1, pack2(c[k], c[k + 1]));
    unpack2(fma2(s2, d2, u2), c[k], c[k + 1]);
  }
}

// One logical row: conditional array, optional unconditional array, optional
// top-k threshold.  Loads VEC consecutive logits starting at element x0.
template <typename T, bool CFG>
struct Row {
  const T* cond;
  const T* uncond;
  float scale;
  float thr;  // entries below thr become -inf (thr = -inf: no filter)
#ifdef CSD_CHECKED
  int n = 0x7fffffff;   // elements in the row (checked build only)
#endif
  static constexpr int kVec = Elem<T>::kVec;

  __device__ __forceinline__ void load_vec(int x0, float (&z)[Elem<T>::kVec]) const {
#ifdef CSD_CHECKED
    if (!checked_ok(x0, kVec, n, 1)) {
#pragma unroll
      for (int k = 0; k < kVec; ++k) z[k] = CSD_NEG_INF;
      return;
    }
#endif
    Elem<T>::load_vec(cond + x0, z);
    if (CFG) {
      float u[kVec];
      Elem<T>::load_vec(uncond + x0, u);
      cfg_mix_vec<kVec>(z, u, scale);
    }
  }
  __device__ __forceinline__ float load_one(int x) const {
#ifdef CSD_CHECKED
    if (!checked_ok(x, 1, n, 2)) return CSD_NEG_INF;
#endif
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
#ifdef CSD_CHECKED
    row.n = a.V;
#endif
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
#ifdef CSD_CHECKED
    row.n = a.V;
#endif
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
  float* diag_am;   // [B, gamma] or null: sum_x Q f per position (inner sum of Eq. token_exp)
  float* diag_bt;   // [B, gamma] or null: bracket of Eq. bd2 per position
  // similarity relaxation (LANTERN++'s acceptance with the paper's G*; multi-launch path only)
  const int32_t* nbr;   // [V, nbr_k] or null: every token's nearest tokens, nearest first (-1: none)
  int nbr_k;
  float nbr_lambda;
  int nbr_table_off;    // > 0: the block's dynamic shared memory has room for a float[V] table of the target's
                        //      probabilities at this offset (in doubles, after the tile sums); 0: look them up in global memory
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
  // P - Q; written with the rounding intrinsics so that no product is contracted into a fused
  // multiply-add: identical rows must give exactly 0 at every call site
  const float pq = __fmul_rn(__fadd_rn(__fsub_rn(et, ed), __fsub_rn(__fmul_rn(et, c.Sd), __fmul_rn(ed, c.St))), c.inv_den);
  const float alt = c.one_minus_omega * et * c.inv_t;                    // (1 - omega) P
  return fmaxf(0.0f, fmaxf(pq, alt));
}

// weight_of for two candidates at once, two values per instruction: the same operations in the same
// order, each half the IEEE operation, so the results are weight_of's bit for bit (a - b is taken as
// fma(b, -1, a), which rounds once like the subtraction).
__device__ __forceinline__ void weight_of_pair(float zt0, float zt1, float zd0, float zd1, const PairCtx& c, float& g0, float& g1) {
  const uint64_t l2e = pack2(kLog2e, kLog2e), m1 = pack2(-1.0f, -1.0f);
  float xt0, xt1;
  unpack2(mul2(add2(pack2(zt0, zt1), pack2(-c.Mt, -c.Mt)), l2e), xt0, xt1);
  const uint64_t et = pack2(ex2f(xt0), ex2f(xt1));
  if (c.mode == 1) {
    unpack2(mul2(et, pack2(c.inv_t, c.inv_t)), g0, g1);
    return;
  }
  float xd0, xd1;
  unpack2(mul2(add2(pack2(zd0, zd1), pack2(-c.Md, -c.Md)), l2e), xd0, xd1);
  const uint64_t ed = pack2(ex2f(xd0), ex2f(xd1));
  const uint64_t diff = fma2(ed, m1, et);                                                   // et - ed
  const uint64_t cross = fma2(mul2(ed, pack2(c.St, c.St)), m1, mul2(et, pack2(c.Sd, c.Sd)));   // et Sd - ed St
  float pq0, pq1, a0, a1;
  unpack2(mul2(add2(diff, cross), pack2(c.inv_den, c.inv_den)), pq0, pq1);
  unpack2(mul2(mul2(pack2(c.one_minus_omega, c.one_minus_omega), et), pack2(c.inv_t, c.inv_t)), a0, a1);
  g0 = fmaxf(0.0f, fmaxf(pq0, a0));
  g1 = fmaxf(0.0f, fmaxf(pq1, a1));
}

// Similarity relaxation (LANTERN++'s P^{k,lambda} at the candidate): the target mass of the selected
// subset of token x's nearest tokens -- taken nearest first while the running sum stays strictly below
// lambda P(x); the first that would break it ends the selection -- to be added to P(x) = own.
template <typename RowT>
__device__ __forceinline__ float neighbour_extra(const RowT& rt, const float Mt, const float inv_t, const int32_t* nbr,
                                                 const int k, const float lambda, const int x, const int V, const float own) {
  float extra = 0.0f;
  const float budget = lambda * own;
  for (int j = 0; j < k; ++j) {
    const int y = __ldg(nbr + (int64_t)x * k + j);
    if (y < 0 || y >= V || y == x) continue;
    const float py = ex2f((rt.filter(rt.load_one(y)) - Mt) * kLog2e) * inv_t;
    if (extra + py < budget) extra += py;
    else break;
  }
  return extra;
}
// The same selection with the target's probabilities read from a table (shared memory).
__device__ __forceinline__ float neighbour_extra_table(const float* tP, const int32_t* nbr, const int k, const float lambda,
                                                       const int x, const int V, const float own) {
  float extra = 0.0f;
  const float budget = lambda * own;
  for (int j = 0; j < k; ++j) {
    const int y = __ldg(nbr + (int64_t)x * k + j);
    if (y < 0 || y >= V || y == x) continue;
    const float py = tP[y];
    if (extra + py < budget) extra += py;
    else break;
  }
  return extra;
}
// Eq. opt_G's weight with that acceptance, g = [P - min{Q, omega (P + extra)}]_+; P - Q in the
// cancellation-free form of weight_of.
__device__ __forceinline__ float weight_of_similar(float zt, float zd, const PairCtx& c, const float extra) {
  const float et = ex2f((zt - c.Mt) * kLog2e), ed = ex2f((zd - c.Md) * kLog2e);
  const float pq = __fmul_rn(__fadd_rn(__fsub_rn(et, ed), __fsub_rn(__fmul_rn(et, c.Sd), __fmul_rn(ed, c.St))), c.inv_den);
  const float P = et * c.inv_t, Q = ed / (1.0f + c.Sd);
  const float oa = (1.0f - c.one_minus_omega) * (P + extra);
  return oa >= Q ? fmaxf(0.0f, pq) : fmaxf(0.0f, P - oa);
}

// One candidate token's share of the two per-position sums of Theorem 2, with
// f(x) = min{1, omega P(x)/Q(x)}: Q f = min{Q, omega P}, and, since sum_x (P - Q f) = sum_x (1 - f) Q,
// the bracket of Eq. bd2 is 2 sum_x [Q f - P]_+.  am and bt2 accumulate sum_x Q f and sum_x [Q f - P]_+.
struct TermsCtx {
  float Mt, Md, inv_t, inv_d, omega;
};
__device__ __forceinline__ void terms_of(float zt, float zd, const TermsCtx& c, float& am, float& bt2) {
  const float P = ex2f((zt - c.Mt) * kLog2e) * c.inv_t;
  const float Q = ex2f((zd - c.Md) * kLog2e) * c.inv_d;
  const float qf = fminf(Q, c.omega * P);
  am += qf;
  bt2 += fmaxf(qf - P, 0.0f);
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

// ---- inverse-CDF draw over per-tile sums (one warp) ---------------------------------------------
// Finds the tile that holds the crossing C(x) > u Z and the sum of the tiles before it; if no tile
// qualifies (u >= 1 or NaN, or rounding), the last tile with positive mass -- the documented rule
// "else the last token with positive weight".  Writes sm.Z, sm.pick_tile (-1: no tile has mass)
// and sm.pick_prefix; every lane of the calling warp takes part.
// With target_abs given, the crossing looked for is C(x) > *target_abs (a vocabulary shard's share of a
// draw whose total is known from all shards) instead of u times this array's own total.
__device__ __forceinline__ void locate_crossing_tile(const double* tile_sums, const int ntiles, const float u,
                                                     const int lane, FinishSmem& sm,
                                                     const double* target_abs = nullptr) {
  const int chunk = (ntiles + 31) / 32;
  const int t0 = min(ntiles, lane * chunk), t1 = min(ntiles, t0 + chunk);
  double local = 0.0;
  for (int t = t0; t < t1; ++t) local += tile_sums[t];
  const double incl = warp_incl_scan_double(local, lane);
  const double Z = __shfl_sync(0xffffffffu, incl, 31);
  const double target = target_abs ? *target_abs : (double)u * Z;
  const unsigned crossing = __ballot_sync(0xffffffffu, incl > target && local > 0.0);
  const unsigned has_mass = __ballot_sync(0xffffffffu, local > 0.0);
  if (lane == 0) { sm.Z = Z; sm.pick_tile = -1; sm.pick_prefix = 0.0; }
  __syncwarp();
  const unsigned from = crossing ? crossing : has_mass;
  if (from == 0) return;
  const int owner = crossing ? __ffs(crossing) - 1 : 31 - __clz(has_mass);
  if (lane == owner) {
    double c = incl - local, c_pick = c;
    int pick = -1;
    for (int t = t0; t < t1; ++t) {
      const double v = tile_sums[t];
      if (v > 0.0) { pick = t; c_pick = c; }   // last tile with mass seen so far
      if (crossing && c + v > target && v > 0.0) break;
      c += v;
    }
    sm.pick_tile = pick;
    sm.pick_prefix = c_pick;
  }
}

// The token inside the picked tile (one warp; lane holds the weights g[0..VEC) of its VEC consecutive
// tokens starting at x0): the first token whose running sum exceeds u Z, else the tile's last token
// with positive weight, else -1.
template <int VEC>
__device__ __forceinline__ int pick_in_tile(const float (&g)[VEC], const int x0, const double prefix,
                                            const double target, const int lane) {
  double run[VEC];
  double acc = 0.0;
  int last_pos = -1;
  unsigned posmask = 0;
#pragma unroll
  for (int k = 0; k < VEC; ++k) {
    if (g[k] > 0.0f) { last_pos = k; posmask |= 1u << k; }
    acc += (double)g[k];
    run[k] = acc;
  }
  const double before = prefix + (warp_incl_scan_double(acc, lane) - acc);
  int first = -1;
#pragma unroll
  for (int k = VEC - 1; k >= 0; --k)
    if (before + run[k] > target && ((posmask >> k) & 1u)) first = k;
  const unsigned hit = __ballot_sync(0xffffffffu, first >= 0);
  const unsigned pos = __ballot_sync(0xffffffffu, last_pos >= 0);
  int token = -1;
  if (hit != 0) token = __shfl_sync(0xffffffffu, x0 + first, __ffs(hit) - 1);
  else if (pos != 0) token = __shfl_sync(0xffffffffu, x0 + last_pos, 31 - __clz(pos));
  return token;
}

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
// double per tile of 32 * (16 bytes / element size) tokens, and at least two per warp.
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
          Row<T, CFG> rt{tgt + (int64_t)i * V, CFG ? tgt_u + (int64_t)i * V : nullptr, a.cfg_scale, thr[0] CSD_ROW_LEN(V)};
          Row<T, CFG> rd{dft + (int64_t)i * V, CFG ? dft_u + (int64_t)i * V : nullptr, a.cfg_scale, thr[1] CSD_ROW_LEN(V)};
          const float dt = rt.filter(rt.load_one(tok)) - M[0];
          const float dd = rd.filter(rd.load_one(tok)) - M[1];
          p = ex2f(dt * kLog2e) / (1.0f + S[0]);
          q = ex2f(dd * kLog2e) / (1.0f + S[1]);
          float grow = 1.0f;   // (aggregated mass) / (own mass) under the similarity relaxation
          if (a.nbr && p > 0.0f) {
            const float extra = neighbour_extra(rt, M[0], 1.0f / (1.0f + S[0]), a.nbr, a.nbr_k, a.nbr_lambda, tok, V, p);
            grow = 1.0f + extra / p;
            p += extra;
          }
          if (dd == CSD_NEG_INF) f = 1.0f;         // q = 0: p/q = +inf, and 0/0 := 1
          else if (dt == CSD_NEG_INF) f = 0.0f;    // p = 0 < q
          else f = fminf(1.0f, omega * grow * ex2f((dt - dd) * kLog2e) * ((1.0f + S[1]) / (1.0f + S[0])));
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
    Row<T, CFG> rt{tgt + (int64_t)j * V, CFG ? tgt_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[0][j] CSD_ROW_LEN(V)};
    Row<T, CFG> rd = rt;
    if (j < L) rd = Row<T, CFG>{dft + (int64_t)j * V, CFG ? dft_u + (int64_t)j * V : nullptr, a.cfg_scale, sm.thr[1][j] CSD_ROW_LEN(V)};
    const float u = a.uniforms[(int64_t)b * (L + 1) + L];
    // (omega >= 1: the aggregated mass only raises f above f_van, and Eq. opt_G is the vanilla residual)
    const bool similar = a.nbr != nullptr && j < L && omega < 1.0f && ctx.mode == 0;
    // Every candidate with target mass then needs the mass of up to k neighbours: where the block's shared
    // memory has room, the target's probabilities are tabulated there once (the same expression, hence the
    // same bits, as a lookup in global memory would evaluate) and the lookups stay on the SM.
    float* const tP = (similar && a.nbr_table_off > 0) ? reinterpret_cast<float*>(tile_sums + a.nbr_table_off) : nullptr;
    if (tP) {
      for (int tile = warp; tile < ntiles; tile += NT / 32) {
        const int x0 = tile * TILE + lane * VEC;
        float zt[VEC];
        rt.load_tile(x0, V, a.vec_ok, zt);
#pragma unroll
        for (int k = 0; k < VEC; ++k)
          if (x0 + k < V) tP[x0 + k] = ex2f((rt.filter(zt[k]) - ctx.Mt) * kLog2e) * ctx.inv_t;
      }
      group_sync<NT, BAR>();
    }
    auto weight_at = [&](int x, float zt_x, float zd_x) -> float {
      const float ft = rt.filter(zt_x);
      if (ctx.mode != 0) return weight_of(ft, 0.0f, ctx);
      const float fd = rd.filter(zd_x);
      if (!similar || x >= V) return weight_of(ft, fd, ctx);
      const float own = ex2f((ft - ctx.Mt) * kLog2e) * ctx.inv_t;
      float extra = 0.0f;
      if (own > 0.0f)
        extra = tP ? neighbour_extra_table(tP, a.nbr, a.nbr_k, a.nbr_lambda, x, V, own)
                   : neighbour_extra(rt, ctx.Mt, ctx.inv_t, a.nbr, a.nbr_k, a.nbr_lambda, x, V, own);
      return weight_of_similar(ft, fd, ctx, extra);
    };

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
            const int x0 = tile * TILE + lane * VEC;
            float acc = 0.0f;
#pragma unroll
            for (int k = 0; k < VEC; ++k)
              acc += weight_at(x0 + k, zt[r][k], ctx.mode == 0 ? zd[r][k] : 0.0f);
            const double tsum = warp_sum_double((double)acc);
            if (lane == 0) tile_sums[tile] = tsum;
          }
        }
      }
      group_sync<NT, BAR>();
      // ---- 5. locate the tile that holds the crossing C(x) > u Z ------------------
      if (warp == 0) locate_crossing_tile(tile_sums, ntiles, u, lane, sm);
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
        int tok = -1;
        if (tile >= 0) {   // (the same decision in every lane)
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC], g[VEC];
          rt.load_tile(x0, V, a.vec_ok, zt);
          if (ctx.mode == 0) rd.load_tile(x0, V, a.vec_ok, zd);
#pragma unroll
          for (int k = 0; k < VEC; ++k)
            g[k] = weight_at(x0 + k, zt[k], ctx.mode == 0 ? zd[k] : 0.0f);
          tok = pick_in_tile<VEC>(g, x0, sm.pick_prefix, (double)u * Z, lane);
        }
        if (lane == 0) sm.token = tok;
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
              G_out[x0 + k] = weight_at(x0 + k, zt[k], ctx.mode == 0 ? zd[k] : 0.0f) * invZ;
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
    if (a.out_accept_len) a.out_accept_len[b] = tau;
    if (a.out_status) a.out_status[b] = status;
  }
  // ---- 9. optional: the per-position sums of Theorem 2 (a second pass over every row) ------------
  if (a.diag_am || a.diag_bt) {
    for (int i = 0; i < L; ++i) {
      group_sync<NT, BAR>();
      float am = 0.0f, bt2 = 0.0f;
      const bool usable = sm.valid[0][i] && sm.valid[1][i];
      if (usable) {
        TermsCtx tc;
        tc.Mt = sm.M[0][i]; tc.Md = sm.M[1][i];
        tc.inv_t = 1.0f / (1.0f + sm.S[0][i]); tc.inv_d = 1.0f / (1.0f + sm.S[1][i]);
        const float om = a.schedule[i];
        tc.omega = om >= 0.0f ? om : 0.0f;
        const Row<T, CFG> rt{tgt + (int64_t)i * V, CFG ? tgt_u + (int64_t)i * V : nullptr, a.cfg_scale, sm.thr[0][i] CSD_ROW_LEN(V)};
        const Row<T, CFG> rd{dft + (int64_t)i * V, CFG ? dft_u + (int64_t)i * V : nullptr, a.cfg_scale, sm.thr[1][i] CSD_ROW_LEN(V)};
        for (int tile = warp; tile < (V + TILE - 1) / TILE; tile += NT / 32) {
          const int x0 = tile * TILE + lane * VEC;
          float zt[VEC], zd[VEC];
          rt.load_tile(x0, V, a.vec_ok, zt);
          rd.load_tile(x0, V, a.vec_ok, zd);
#pragma unroll
          for (int k = 0; k < VEC; ++k)
            if (x0 + k < V) terms_of(rt.filter(zt[k]), rd.filter(zd[k]), tc, am, bt2);
        }
      }
      const double wa = warp_sum_double((double)am), wb = warp_sum_double((double)bt2);
      if (lane == 0) { tile_sums[2 * warp] = wa; tile_sums[2 * warp + 1] = wb; }
      group_sync<NT, BAR>();
      if (tid == 0) {
        double ta = 0.0, tb = 0.0;
        for (int w = 0; w < NT / 32; ++w) { ta += tile_sums[2 * w]; tb += tile_sums[2 * w + 1]; }
        const float nanv = __int_as_float(0x7fc00000);
        if (a.diag_am) a.diag_am[(int64_t)b * L + i] = usable ? (float)ta : nanv;
        if (a.diag_bt) a.diag_bt[(int64_t)b * L + i] = usable ? (float)(2.0 * tb) : nanv;
      }
    }
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

}  // namespace csd
