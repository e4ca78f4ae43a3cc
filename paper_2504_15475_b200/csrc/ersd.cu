// libersd: exponential-race speculative decoding kernels for sm_100a and their C entry points.
//
// One thread block streams one chunk of one logit row (or of a draft/target
// row pair that shares its race variables).  Per vocabulary index it draws the
// 32-bit Philox word, forms a cheap single-precision screening key and keeps
// only the indices that can still be among the first c arrivals; those few
// are re-evaluated in double precision and inserted into a per-warp sorted
// list.  Lists are merged per block, exchanged through a small workspace, and
// the last block of a sequence turns the winners into the accepted prefix
// (sequence scan or tree walk) in the same launch.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "ersd.h"
#include "ersd_math.cuh"

namespace ersd {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPerThread = 8;
constexpr int kTile = kThreads * kPerThread;  // vocabulary indices per block iteration
constexpr int kPartCap = 64;                  // partial-list entries per (row, role) in the workspace
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct Entry {  // one arrival: race key (natural-log units) and token id
  double key;
  int32_t idx;
  int32_t pad;
};

// Workspace layout: one slot per logit row, whatever the call's sizes, so that a counter field
// is never reused as a partial-list field by a later call with other sizes (counters must be
// zero when a call starts; partial lists are always rewritten before they are read).
struct Slot {
  int counter;  // arrivals of the group whose first row this is; reset to 0 by the last arrival
  int pad[3];
  Entry part[2][kPartCap];  // per role: S partial lists of c entries each
};

struct TreeDesc {  // draft tree of one call, passed by value in kernel parameter space
  int16_t parent[ERSD_MAX_ROWS];
  int16_t first_child[ERSD_MAX_ROWS];
  int16_t next_sib[ERSD_MAX_ROWS];
  uint8_t rank[ERSD_MAX_ROWS];
  uint8_t nchild[ERSD_MAX_ROWS];
  uint8_t order[ERSD_MAX_ROWS];  // launch order of rows: rows with a draft row first
};

enum Mode { kSample = 0, kVerify = 1 };

struct Params {
  const void* target;  // target logits (race_sample: the logits)
  const void* draft;
  int64_t ld_t, ld_d;
  const uint64_t* seeds;
  const uint32_t* seq_ids;
  const uint32_t* pos_offsets;
  const float* temps;
  int64_t ts_b, ts_r;
  float T;
  int B, rows, V;
  int S, per_chunk;
  int mode;
  int c_sample;          // arrivals per row in sample mode
  int draft_rows;        // draft rows per sequence (k, or N + 1 for trees)
  int depth;             // columns of out_tokens - 1
  int chain_outputs;     // 1: out_draft_* are [B, k] indexed by position (sequence variant)
  int aligned_t, aligned_d;
  int32_t* out_tokens;
  int32_t* out_accept_len;
  int32_t* out_path;
  int32_t* out_draft_tok;
  float* out_draft_key;
  int32_t* out_target_tok;
  float* out_target_key;
  float* out_key;        // sample mode
  Slot* slots;
};

// ---------------------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int ord_of(float f) {  // monotone float -> int map
  int o = __float_as_int(f);
  return o ^ ((o >> 31) & 0x7FFFFFFF);
}
__device__ __forceinline__ float float_of(int o) { return __int_as_float(o ^ ((o >> 31) & 0x7FFFFFFF)); }

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

template <int DT>
struct Raw;
template <>
struct Raw<ERSD_BF16> {
  uint4 a;
};
template <>
struct Raw<ERSD_F32> {
  uint4 a, b;
};

// Eight logits starting at element i0 of a row; elements at or beyond `vend` read as NaN.
template <int DT>
__device__ __forceinline__ Raw<DT> fetch(const void* row, int i0, int vend, bool aligned) {
  Raw<DT> r;
  if constexpr (DT == ERSD_BF16) {
    const uint16_t* p = (const uint16_t*)row;
    if (aligned && i0 + kPerThread <= vend) {
      r.a = ldg_stream(p + i0);
    } else {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int e0 = i0 + 2 * j, e1 = e0 + 1;
        const uint32_t lo = (e0 < vend) ? (uint32_t)__ldg(p + e0) : 0x7FC0u;
        const uint32_t hi = (e1 < vend) ? (uint32_t)__ldg(p + e1) : 0x7FC0u;
        w[j] = lo | (hi << 16);
      }
      r.a = make_uint4(w[0], w[1], w[2], w[3]);
    }
  } else {
    const uint32_t* p = (const uint32_t*)row;
    if (aligned && i0 + kPerThread <= vend) {
      r.a = ldg_stream(p + i0);
      r.b = ldg_stream(p + i0 + 4);
    } else {
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = (i0 + j < vend) ? __ldg(p + i0 + j) : 0x7FC00000u;
      r.a = make_uint4(w[0], w[1], w[2], w[3]);
      r.b = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
  return r;
}

__device__ __forceinline__ void decode(const Raw<ERSD_BF16>& r, float z[8]) {
  const uint32_t w[4] = {r.a.x, r.a.y, r.a.z, r.a.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    z[2 * j] = __uint_as_float(w[j] << 16);
    z[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void decode(const Raw<ERSD_F32>& r, float z[8]) {
  z[0] = __uint_as_float(r.a.x); z[1] = __uint_as_float(r.a.y);
  z[2] = __uint_as_float(r.a.z); z[3] = __uint_as_float(r.a.w);
  z[4] = __uint_as_float(r.b.x); z[5] = __uint_as_float(r.b.y);
  z[6] = __uint_as_float(r.b.z); z[7] = __uint_as_float(r.b.w);
}

// Sorted list of the smallest (key, idx) pairs seen by a warp: lane l holds the l-th smallest.
struct WarpList {
  double key;
  int idx;
  __device__ __forceinline__ void init() {
    key = (double)INFINITY;
    idx = 0x7FFFFFFF;
  }
  // warp-uniform arguments; keeps ascending (key, idx) order
  __device__ __forceinline__ void insert(double k, int i, int lane) {
    const bool before = (key < k) || (key == k && idx < i);
    const int pos = __popc(__ballot_sync(kFull, before));
    const double pk = __shfl_up_sync(kFull, key, 1);
    const int pi = __shfl_up_sync(kFull, idx, 1);
    if (lane > pos) {
      key = pk;
      idx = pi;
    } else if (lane == pos) {
      key = k;
      idx = i;
    }
  }
  __device__ __forceinline__ double key_at(int l) const { return __shfl_sync(kFull, key, l); }
};

// Upper bound, in the screening keys' log2 units, of a double key in natural-log units.
__device__ __forceinline__ float tau_of_exact(double key) {
  const float t = (float)(key * 1.4426950408889634);
  return fmaf(fabsf(t), 2.384185791015625e-7f, t);
}

// c-th smallest of the lanes' values (c >= 1), +inf if fewer than c lanes hold a number.
__device__ __forceinline__ float cth_smallest(float m, int c, int lane) {
  int o = (m == m) ? ord_of(m) : 0x7FFFFFFF;
  int v = 0x7FFFFFFF;
  for (int r = 0; r < c; ++r) {
    v = __reduce_min_sync(kFull, o);
    if (r + 1 == c) break;
    const unsigned eq = __ballot_sync(kFull, o == v);
    if (lane == __ffs(eq) - 1) o = 0x7FFFFFFF;
  }
  return (v == 0x7FFFFFFF) ? INFINITY : float_of(v);
}

// State of one role (target row or draft row) of the block's work item.
struct Role {
  const void* row;
  bool aligned;
  int c;        // arrivals wanted
  float tau;    // log2 units: no index whose true key exceeds tau can be among the first c
  WarpList list;
};

// Shared-memory float minimum (rare path).
__device__ __forceinline__ void smem_min(float* addr, float v) {
  float old = *(volatile float*)addr;
  while (v < old) {
    const float seen = __int_as_float(atomicCAS((int*)addr, __float_as_int(old), __float_as_int(v)));
    if (seen == old) break;
    old = seen;
  }
}

// Upper bound of the eight logits of a tile slice (NaN ignored; NaN if all are NaN).
__device__ __forceinline__ float logits_upper_bound(const Raw<ERSD_BF16>& r) {
  uint32_t m01, m23, m;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(m01) : "r"(r.a.x), "r"(r.a.y));
  asm("max.bf16x2 %0, %1, %2;" : "=r"(m23) : "r"(r.a.z), "r"(r.a.w));
  asm("max.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(m01), "r"(m23));
  // The odd elements' maximum sits in the high half.  Read with the low half attached it is
  // off by less than one bf16 ulp (2^-7 relative, towards larger magnitude); widen it to a
  // sure upper bound instead of masking.
  const float hi_raw = __uint_as_float(m);
  const float hi_ub = fmaf(fabsf(hi_raw), 0.0078125f, hi_raw);
  const float lo = __uint_as_float(m << 16);
  return fmaxf(hi_ub, lo);
}
__device__ __forceinline__ float logits_upper_bound(const Raw<ERSD_F32>& r) {
  const float a = fmaxf(fmaxf(__uint_as_float(r.a.x), __uint_as_float(r.a.y)),
                        fmaxf(__uint_as_float(r.a.z), __uint_as_float(r.a.w)));
  const float b = fmaxf(fmaxf(__uint_as_float(r.b.x), __uint_as_float(r.b.y)),
                        fmaxf(__uint_as_float(r.b.z), __uint_as_float(r.b.w)));
  return fmaxf(a, b);
}

// Examine eight indices of one role: a[j] = lg[j] - z[j] * c2 is either the screening key
// (`accurate`: within the slack of the true key, so the c-th smallest lane minimum also
// tightens tau) or only a lower bound of it.  Indices that can still be among the first c
// arrivals are evaluated in double precision and inserted into the warp's list.
__device__ __forceinline__ void race_role(Role& R, const float z[8], const float lg[8],
                                          const uint32_t xs[8], int i0, float c2, float T,
                                          float* sm_tau, int lane, bool accurate) {
  float a[8];
  float m = INFINITY;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    a[j] = fmaf(-z[j], c2, lg[j]);
    m = fminf(m, a[j]);
  }
  const float tau_in = fminf(R.tau, *(volatile float*)sm_tau);
  float tau = tau_in;
  const bool hit = m <= tau + screen_slack(tau);
  if (__any_sync(kFull, hit)) {
    if (accurate) {
      const float theta = cth_smallest(m, R.c, lane);
      tau = fminf(tau, theta + screen_slack(theta));
    }
    const float lim = tau + screen_slack(tau);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool cand = a[j] <= lim;
      if (__any_sync(kFull, cand)) {
        double dk = (double)INFINITY;
        if (cand) dk = exact_key(xs[j], z[j], T);
        unsigned act = __ballot_sync(kFull, cand && dk < (double)INFINITY);
        while (act) {
          const int src = __ffs(act) - 1;
          act &= act - 1;
          const double k = __shfl_sync(kFull, dk, src);
          const int i = __shfl_sync(kFull, i0, src) + j;
          R.list.insert(k, i, lane);
        }
      }
    }
    const double kc = R.list.key_at(R.c - 1);
    if (kc < (double)INFINITY) tau = fminf(tau, tau_of_exact(kc));
    if (lane == 0 && tau < tau_in) smem_min(sm_tau, tau);
  }
  R.tau = tau;
}

// Stream one chunk [v0, v1) of a row (NR = 1) or of a draft/target pair (NR = 2).
//
// Fast path per thread and tile of eight indices: two Philox calls, the smallest of the eight
// words, the largest of the eight logits per role, and one comparison per role of
//     lg2(x_min) - z_max * c2      (a lower bound of all eight keys, shifted by 32)
// against the block's threshold.  Only when some lane of the warp cannot rule its eight
// indices out does the warp look at them one by one (race_role).
template <int DT, int NR>
__device__ __forceinline__ void stream_chunk(Role* roles, int v0, int v1, const PhiloxRow& pr,
                                             float c2, float T, bool greedy, float* sm_tau,
                                             int lane) {
  const int tid = threadIdx.x;
  const int ntiles = (v1 - v0 + kTile - 1) / kTile;
  Raw<DT> cur[NR], nxt[NR];
  int i0 = v0 + tid * kPerThread;
#pragma unroll
  for (int r = 0; r < NR; ++r) cur[r] = fetch<DT>(roles[r].row, i0, v1, roles[r].aligned);
  for (int t = 0; t < ntiles; ++t) {
    const int in = i0 + kTile;
    if (t + 1 < ntiles) {
#pragma unroll
      for (int r = 0; r < NR; ++r) nxt[r] = fetch<DT>(roles[r].row, in, v1, roles[r].aligned);
    }
    uint32_t xs[8];
    pr.words((uint32_t)i0 >> 2, xs);
    pr.words(((uint32_t)i0 >> 2) + 1u, xs + 4);
    const uint32_t xm = min(min(min(xs[0], xs[1]), min(xs[2], xs[3])),
                            min(min(xs[4], xs[5]), min(xs[6], xs[7])));
    // lg2(w) >= lg2(x) - 32; the 32 moves to the threshold's side.  Greedy rows have no race.
    const float lgm = greedy ? 32.0f : lg2_fast((float)xm);
    bool pass = false, boot = false;
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const float tau = *(volatile float*)(sm_tau + r);
      const float lim32 = fmaf(fabsf(tau), 9.5367431640625e-7f, tau) + 32.001953125f;
      const float lb = fmaf(-logits_upper_bound(cur[r]), c2, lgm);
      pass |= !(lb > lim32);
      boot |= !(tau < INFINITY);
    }
    if (__any_sync(kFull, pass)) {
      // No threshold yet (first tiles of a chunk): use the accurate screening value so that
      // the tile itself yields one.  Otherwise the cheaper lower bound lg2(x) - 32 will do.
      float lg[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        lg[j] = greedy ? 0.0f : (boot ? screen_lg2_e(xs[j]) : lg2_fast((float)xs[j]) - 32.0f);
#pragma unroll
      for (int r = 0; r < NR; ++r) {
        float z[8];
        decode(cur[r], z);
        race_role(roles[r], z, lg, xs, i0, c2, T, sm_tau + r, lane, boot || greedy);
      }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) cur[r] = nxt[r];
    i0 = in;
  }
}

// Merge `n` sorted partial lists of `c` entries each (global memory written by other blocks)
// into a fresh warp list.
__device__ __forceinline__ void merge_partials(WarpList& L, const Entry* part, int n, int c,
                                               int lane) {
  L.init();
  for (int e = 0; e < n * c; ++e) {
    const double k = __ldcg(&part[e].key);
    const int i = __ldcg(&part[e].idx);
    if (i != 0x7FFFFFFF) L.insert(k, i, lane);  // unused slots carry idx = INT_MAX
  }
}

#ifndef ERSD_MIN_BLOCKS
#define ERSD_MIN_BLOCKS 2  // resident blocks per SM the register allocation aims for
#endif

template <int DT>
__global__ void __launch_bounds__(kThreads, ERSD_MIN_BLOCKS)
ersd_race_kernel(const Params p, const __grid_constant__ TreeDesc tree) {
  __shared__ float sm_tau[2];
  __shared__ Entry sm_list[2][kWarps][ERSD_MAX_TOP_C];
  __shared__ int sm_last;
  __shared__ int sm_ttok[ERSD_MAX_ROWS], sm_dtok[ERSD_MAX_ROWS];
  __shared__ float sm_tkey[ERSD_MAX_ROWS], sm_dkey[ERSD_MAX_ROWS];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // work item -> (row, sequence, chunk); rows are launched in tree.order so that the heavier
  // paired rows start first
  const int per_row = p.B * p.S;
  const int ri = blockIdx.x / per_row;
  const int rem = blockIdx.x - ri * per_row;
  const int b = rem / p.S;
  const int s = rem - b * p.S;
  const int r = (p.mode == kSample) ? ri : (int)tree.order[ri];
  const int unit = b * p.rows + r;

  const int cq = (p.mode == kSample) ? 0 : (int)tree.nchild[r];
  const int c0 = (p.mode == kSample) ? p.c_sample : 1;
  const int v0 = s * p.per_chunk;
  const int v1 = min(p.V, v0 + p.per_chunk);

  const uint64_t seed = p.seeds[b];
  const uint32_t seq = p.seq_ids ? p.seq_ids[b] : (uint32_t)b;
  const uint32_t pos = (p.pos_offsets ? p.pos_offsets[b] : 0u) + (uint32_t)r;
  const float T = p.temps ? p.temps[(int64_t)b * p.ts_b + (int64_t)r * p.ts_r] : p.T;
  const bool greedy = (T == 0.0f);
  float c2;
  if (greedy) c2 = 1.0f;
  else if (T > 0.0f && T < INFINITY) c2 = (float)(1.4426950408889634 / (double)T);
  else c2 = __int_as_float(0x7FC00000);  // invalid temperature: no token arrives

  if (tid < 2) sm_tau[tid] = INFINITY;
  __syncthreads();
  PhiloxRow pr;
  pr.init(seed, seq, pos);

  const size_t es = (DT == ERSD_BF16) ? 2 : 4;
  Role roles[2];
  roles[0].row = (const char*)p.target + (size_t)unit * (size_t)p.ld_t * es;
  roles[0].aligned = p.aligned_t;
  roles[0].c = c0;
  roles[0].tau = INFINITY;
  roles[0].list.init();
  roles[1].row = nullptr;
  roles[1].aligned = p.aligned_d;
  roles[1].c = cq > 0 ? cq : 1;
  roles[1].tau = INFINITY;
  roles[1].list.init();
  if (cq > 0) {
    roles[1].row = (const char*)p.draft + ((size_t)b * p.draft_rows + r) * (size_t)p.ld_d * es;
    stream_chunk<DT, 2>(roles, v0, v1, pr, c2, T, greedy, sm_tau, lane);
  } else {
    stream_chunk<DT, 1>(roles, v0, v1, pr, c2, T, greedy, sm_tau, lane);
  }

  // ---- block merge: every warp publishes its list, warp `role` merges that role's lists ----
  const int nroles = cq > 0 ? 2 : 1;
#pragma unroll
  for (int role = 0; role < 2; ++role) {
    if (role >= nroles) break;
    Entry e;
    e.key = roles[role].list.key;
    e.idx = roles[role].list.idx;
    e.pad = 0;
    sm_list[role][warp][lane] = e;
  }
  __syncthreads();
  const bool direct = (p.mode == kSample && p.S == 1);
  if (warp < nroles) {
    const int role = warp;
    const int c = role ? roles[1].c : roles[0].c;
    WarpList L = role ? roles[1].list : roles[0].list;
    for (int w = 0; w < kWarps; ++w) {
      if (w == warp) continue;
      for (int e = 0; e < c; ++e) {
        const Entry en = sm_list[role][w][e];
        if (en.idx != 0x7FFFFFFF) L.insert(en.key, en.idx, lane);
      }
    }
    if (direct) {
      if (lane < c) {
        const bool ok = L.idx != 0x7FFFFFFF;
        const size_t o = (size_t)unit * c + lane;
        p.out_tokens[o] = ok ? L.idx : -1;
        if (p.out_key) p.out_key[o] = ok ? (float)L.key : INFINITY;
      }
    } else if (lane < c) {
      Entry e;
      e.key = L.key;
      e.idx = L.idx;
      e.pad = 0;
      p.slots[unit].part[role][s * c + lane] = e;
    }
  }
  if (direct) return;

  // ---- the last block of the group (row in sample mode, sequence otherwise) finishes ----
  __threadfence();
  __syncthreads();
  int* counter = &p.slots[(p.mode == kSample) ? unit : b * p.rows].counter;
  const int group_items = (p.mode == kSample) ? p.S : p.rows * p.S;
  if (tid == 0) {
    const int old = atomicAdd(counter, 1);
    sm_last = (old == group_items - 1);
  }
  __syncthreads();
  if (!sm_last) return;
  __threadfence();
  if (tid == 0) *counter = 0;  // leave the workspace ready for the next call

  if (p.mode == kSample) {
    if (warp == 0) {
      WarpList L;
      merge_partials(L, p.slots[unit].part[0], p.S, c0, lane);
      if (lane < c0) {
        const bool ok = L.idx != 0x7FFFFFFF;
        const size_t o = (size_t)unit * c0 + lane;
        p.out_tokens[o] = ok ? L.idx : -1;
        if (p.out_key) p.out_key[o] = ok ? (float)L.key : INFINITY;
      }
    }
    return;
  }

  // verify: final arrivals of every row of sequence b
  for (int combo = warp; combo < p.rows * 2; combo += kWarps) {
    const int n = combo >> 1, role = combo & 1;
    const int c = role ? (int)tree.nchild[n] : 1;
    if (c == 0) continue;
    WarpList L;
    merge_partials(L, p.slots[b * p.rows + n].part[role], p.S, c, lane);
    const bool ok = L.idx != 0x7FFFFFFF;
    if (role == 0) {
      if (lane == 0) {
        sm_ttok[n] = ok ? L.idx : -1;
        sm_tkey[n] = ok ? (float)L.key : INFINITY;
      }
    } else if (lane < c) {
      int m = tree.first_child[n];  // the child of rank `lane`
      for (int q = 0; q < lane; ++q) m = tree.next_sib[m];
      sm_dtok[m] = ok ? L.idx : -1;
      sm_dkey[m] = ok ? (float)L.key : INFINITY;
    }
  }
  if (tid == 0) {
    sm_dtok[0] = -1;
    sm_dkey[0] = INFINITY;
  }
  __syncthreads();

  const int cols = p.depth + 1;
  for (int d = tid; d < cols; d += kThreads) {
    p.out_tokens[(size_t)b * cols + d] = -1;
    if (p.out_path) p.out_path[(size_t)b * cols + d] = -1;
  }
  for (int n = tid; n < p.rows; n += kThreads) {
    const size_t o = (size_t)b * p.rows + n;
    if (p.out_target_tok) p.out_target_tok[o] = sm_ttok[n];
    if (p.out_target_key) p.out_target_key[o] = sm_tkey[n];
    if (p.chain_outputs) {
      if (n >= 1) {
        const size_t od = (size_t)b * (p.rows - 1) + (n - 1);
        if (p.out_draft_tok) p.out_draft_tok[od] = sm_dtok[n];
        if (p.out_draft_key) p.out_draft_key[od] = sm_dkey[n];
      }
    } else {
      if (p.out_draft_tok) p.out_draft_tok[o] = sm_dtok[n];
      if (p.out_draft_key) p.out_draft_key[o] = sm_dkey[n];
    }
  }
  __syncthreads();
  if (tid == 0) {
    // Walk down from the root while the target winner of the current node's race is the
    // token drafted at one of its children.
    int cur = 0, depth = 0;
    for (;;) {
      const int w = sm_ttok[cur];
      p.out_tokens[(size_t)b * cols + depth] = w;
      if (p.out_path) p.out_path[(size_t)b * cols + depth] = cur;
      int next = -1;
      if (w >= 0) {
        for (int m = tree.first_child[cur]; m >= 0; m = tree.next_sib[m]) {
          if (sm_dtok[m] == w) {
            next = m;
            break;
          }
        }
      }
      if (next < 0 || depth >= p.depth) break;
      cur = next;
      ++depth;
    }
    p.out_accept_len[b] = depth;
  }
}

template <int DT>
__global__ void ersd_row_keys_kernel(const void* row, int V, float T, uint64_t seed, uint32_t seq,
                                     uint32_t pos, int mode, float* out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= V) return;
  float z;
  if (DT == ERSD_BF16) z = __uint_as_float((uint32_t)((const uint16_t*)row)[i] << 16);
  else z = ((const float*)row)[i];
  const uint32_t x = token_word(seed, seq, pos, (uint32_t)i);
  if (mode == 0) {
    out[i] = (float)exact_key(x, z, T);
  } else {
    const float c2 = (T == 0.0f) ? 1.0f : (float)(1.4426950408889634 / (double)T);
    const float lg = (T == 0.0f) ? 0.0f : screen_lg2_e(x);
    out[i] = fmaf(-z, c2, lg) * kLn2;
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static thread_local int g_last_cuda_error = 0;

static int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return ERSD_ECUDA;
}

struct OwnedWorkspace {
  void* ptr = nullptr;
  size_t bytes = 0;
};
static std::mutex g_ws_mutex;
static OwnedWorkspace g_ws[64];

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static size_t workspace_bytes(int64_t B, int64_t rows) {
  return (size_t)B * (size_t)rows * sizeof(Slot);
}

static int get_workspace(const ersd_opts& o, size_t need, void** ws) {
  if (o.workspace) {
    if (o.workspace_bytes < need) return ERSD_EWORKSPACE;
    if (((uintptr_t)o.workspace & 15) != 0) return ERSD_EALIGN;
    *ws = o.workspace;
    return ERSD_OK;
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return ERSD_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  OwnedWorkspace& w = g_ws[dev];
  if (w.bytes < need) {
    if (w.ptr) {
      e = cudaFree(w.ptr);
      w.ptr = nullptr;
      w.bytes = 0;
      if (e != cudaSuccess) return cuda_fail(e);
    }
    const size_t grow = align_up(need + need / 2, 1 << 20);
    e = cudaMalloc(&w.ptr, grow);
    if (e != cudaSuccess) {
      w.ptr = nullptr;
      return cuda_fail(e);
    }
    e = cudaMemset(w.ptr, 0, grow);
    if (e != cudaSuccess) return cuda_fail(e);
    w.bytes = grow;
  }
  *ws = w.ptr;
  return ERSD_OK;
}

static ersd_opts read_opts(const ersd_opts* opts) {
  ersd_opts o;
  memset(&o, 0, sizeof o);
  if (opts) {
    size_t n = opts->struct_size;
    if (n == 0 || n > sizeof o) n = sizeof o;
    memcpy(&o, opts, n);
  }
  return o;
}

static bool temp_ok(float T) { return T >= 0.0f && T < INFINITY; }

static int elem_size(int dt) { return dt == ERSD_BF16 ? 2 : 4; }

static bool rows_aligned(const void* base, int64_t ld, int dt) {
  return ((uintptr_t)base & 15) == 0 && ((ld * elem_size(dt)) & 15) == 0;
}

// Thread blocks per row: enough work items to fill the GPU, chunks of at least four tiles.
static int choose_split(const ersd_opts& o, int64_t units, int V, int cmax) {
  int smax = kPartCap / cmax;
  if (smax > ERSD_MAX_SPLIT) smax = ERSD_MAX_SPLIT;
  const int by_v = (V + 4 * kTile - 1) / (4 * kTile);
  if (smax > by_v) smax = by_v;
  if (smax < 1) smax = 1;
  int S;
  if (o.split_v) {
    S = (int)o.split_v;
  } else {
    const int64_t slots = 148 * 4;
    S = (int)((slots + units - 1) / units);
  }
  if (S > smax) S = smax;
  if (S < 1) S = 1;
  return S;
}

static void set_chunks(Params& p, int S) {
  int per = (p.V + S - 1) / S;
  per = (per + kTile - 1) / kTile * kTile;
  p.per_chunk = per;
  p.S = (p.V + per - 1) / per;
}

static int build_tree(const int32_t* parent, int N, TreeDesc* t, int* depth_out, int* cmax_out) {
  const int nodes = N + 1;
  if (parent[0] != -1) return ERSD_EINVAL;
  int depth[ERSD_MAX_ROWS];
  int last_child[ERSD_MAX_ROWS];
  memset(t, 0, sizeof *t);
  for (int n = 0; n < nodes; ++n) {
    t->first_child[n] = -1;
    t->next_sib[n] = -1;
    last_child[n] = -1;
  }
  t->parent[0] = -1;
  depth[0] = 0;
  int D = 0, cmax = 1;
  for (int n = 1; n < nodes; ++n) {
    const int par = parent[n];
    if (par < 0 || par >= n) return ERSD_EINVAL;
    t->parent[n] = (int16_t)par;
    if (t->nchild[par] >= ERSD_MAX_TOP_C) return ERSD_EUNSUPPORTED;
    t->rank[n] = t->nchild[par]++;
    if (last_child[par] < 0) t->first_child[par] = (int16_t)n;
    else t->next_sib[last_child[par]] = (int16_t)n;
    last_child[par] = n;
    depth[n] = depth[par] + 1;
    if (depth[n] > D) D = depth[n];
    if (t->nchild[par] > cmax) cmax = t->nchild[par];
  }
  int k = 0;
  for (int n = 0; n < nodes; ++n)
    if (t->nchild[n] > 0) t->order[k++] = (uint8_t)n;
  for (int n = 0; n < nodes; ++n)
    if (t->nchild[n] == 0) t->order[k++] = (uint8_t)n;
  *depth_out = D;
  *cmax_out = cmax;
  return ERSD_OK;
}

static int launch(const Params& p, const TreeDesc& tree, int dt, cudaStream_t st) {
  const int64_t items = (int64_t)p.B * p.rows * p.S;
  if (items > 0x7FFFFFFF) return ERSD_EINVAL;
  if (dt == ERSD_BF16) ersd_race_kernel<ERSD_BF16><<<(unsigned)items, kThreads, 0, st>>>(p, tree);
  else ersd_race_kernel<ERSD_F32><<<(unsigned)items, kThreads, 0, st>>>(p, tree);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

static int check_common(const void* logits, int dt, const uint64_t* seeds, int B, int rows, int V,
                        float T) {
  if (!logits || !seeds) return ERSD_EINVAL;
  if (dt != ERSD_F32 && dt != ERSD_BF16) return ERSD_EINVAL;
  if (B < 1 || rows < 1 || V < 1) return ERSD_EINVAL;
  if ((int64_t)B * rows > 0x7FFFFFFF) return ERSD_EINVAL;
  if (V > 0x7FFF0000) return ERSD_EUNSUPPORTED;
  if (!temp_ok(T)) return ERSD_EINVAL;
  if (((uintptr_t)logits & (elem_size(dt) - 1)) != 0 || ((uintptr_t)seeds & 7) != 0)
    return ERSD_EALIGN;
  return ERSD_OK;
}

static void fill_common(Params& p, const ersd_opts& o, const uint64_t* seeds, int B, int rows, int V,
                        float T) {
  p.seeds = seeds;
  p.seq_ids = o.seq_ids;
  p.pos_offsets = o.pos_offsets;
  p.temps = o.temps;
  p.ts_b = o.temp_stride_b;
  p.ts_r = o.temp_stride_r;
  p.T = T;
  p.B = B;
  p.rows = rows;
  p.V = V;
}

static int verify_impl(const void* target, const void* draft, int dt, const TreeDesc& tree, int D,
                       int cmax, bool chain, const uint64_t* seeds, int B, int rows, int draft_rows,
                       int V, float T, int32_t* out_tokens, int32_t* out_accept_len,
                       const ersd_opts* opts, void* stream) {
  const ersd_opts o = read_opts(opts);
  Params p;
  memset(&p, 0, sizeof p);
  fill_common(p, o, seeds, B, rows, V, T);
  p.target = target;
  p.draft = draft;
  p.ld_t = o.ld_target ? o.ld_target : V;
  p.ld_d = o.ld_draft ? o.ld_draft : V;
  if (p.ld_t < V || p.ld_d < V) return ERSD_EINVAL;
  p.mode = kVerify;
  p.c_sample = 1;
  p.draft_rows = draft_rows;
  p.depth = D;
  p.chain_outputs = chain ? 1 : 0;
  p.aligned_t = rows_aligned(target, p.ld_t, dt);
  p.aligned_d = draft ? rows_aligned(draft, p.ld_d, dt) : 1;
  p.out_tokens = out_tokens;
  p.out_accept_len = out_accept_len;
  p.out_path = o.out_path;
  p.out_draft_tok = o.out_draft_tok;
  p.out_draft_key = o.out_draft_key;
  p.out_target_tok = o.out_target_tok;
  p.out_target_key = o.out_target_key;
  set_chunks(p, choose_split(o, (int64_t)B * rows, V, cmax));
  void* ws = nullptr;
  const int st = get_workspace(o, workspace_bytes(B, rows), &ws);
  if (st != ERSD_OK) return st;
  p.slots = (Slot*)ws;
  return launch(p, tree, dt, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Scratch for ersd_verify_noalloc: lives in the library image, one copy per GPU that loads it.
// In host code `g_noalloc_scratch` is only a handle for the runtime, never an address to hand
// to a kernel; noalloc_scratch() asks the runtime for the device address, once per device.
// ---------------------------------------------------------------------------------------------
constexpr size_t kNoallocBytes = (size_t)ERSD_NOALLOC_MAX_ROWS * sizeof(Slot);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocBytes];

static std::mutex g_noalloc_mutex;
static void* g_noalloc_ptr[64];

static int noalloc_scratch(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return ERSD_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);  // address on the current device
    if (e != cudaSuccess) return cuda_fail(e);
    if (!ptr) return ERSD_ECUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  *out = g_noalloc_ptr[dev];
  return ERSD_OK;
}

}  // namespace ersd

using namespace ersd;

extern "C" {

int ersd_race_sample(const void* logits, ersd_dtype dt, const uint64_t* seeds, int B, int R, int V,
                     float T, int32_t* out_tok, const ersd_opts* opts, void* cuda_stream) {
  int st = check_common(logits, dt, seeds, B, R, V, T);
  if (st != ERSD_OK) return st;
  if (!out_tok) return ERSD_EINVAL;
  const ersd_opts o = read_opts(opts);
  const int c = o.top_c > 1 ? (int)o.top_c : 1;
  if (c > ERSD_MAX_TOP_C) return ERSD_EUNSUPPORTED;
  Params p;
  memset(&p, 0, sizeof p);
  fill_common(p, o, seeds, B, R, V, T);
  p.target = logits;
  p.ld_t = o.ld_target ? o.ld_target : V;
  if (p.ld_t < V) return ERSD_EINVAL;
  p.ld_d = V;
  p.mode = kSample;
  p.c_sample = c;
  p.aligned_t = rows_aligned(logits, p.ld_t, dt);
  p.aligned_d = 1;
  p.out_tokens = out_tok;
  p.out_key = o.out_key;
  set_chunks(p, choose_split(o, (int64_t)B * R, V, c));
  if (p.S > 1) {
    void* ws = nullptr;
    st = get_workspace(o, workspace_bytes(B, R), &ws);
    if (st != ERSD_OK) return st;
    p.slots = (Slot*)ws;
  }
  TreeDesc tree;
  memset(&tree, 0, sizeof tree);
  return launch(p, tree, dt, (cudaStream_t)cuda_stream);
}

int ersd_verify(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream) {
  if (k < 0) return ERSD_EINVAL;
  if (k + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  int st = check_common(target_logits, dt, seeds, B, k + 1, V, T);
  if (st != ERSD_OK) return st;
  if (!out_tokens || !out_accept_len) return ERSD_EINVAL;
  if (k > 0) {
    if (!draft_logits) return ERSD_EINVAL;
    if (((uintptr_t)draft_logits & (elem_size(dt) - 1)) != 0) return ERSD_EALIGN;
  }
  int32_t parent[ERSD_MAX_ROWS];
  for (int n = 0; n <= k; ++n) parent[n] = n - 1;
  TreeDesc tree;
  int D = 0, cmax = 1;
  st = build_tree(parent, k, &tree, &D, &cmax);
  if (st != ERSD_OK) return st;
  return verify_impl(target_logits, draft_logits, dt, tree, D, cmax, true, seeds, B, k + 1, k, V, T,
                     out_tokens, out_accept_len, opts, cuda_stream);
}

int ersd_verify_tree(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                     const int32_t* parent, const uint64_t* seeds, int B, int N, int V, float T,
                     int32_t* out_tokens, int32_t* out_accept_len, const ersd_opts* opts,
                     void* cuda_stream) {
  if (N < 0 || !parent) return ERSD_EINVAL;
  if (N + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  int st = check_common(target_logits, dt, seeds, B, N + 1, V, T);
  if (st != ERSD_OK) return st;
  if (!out_tokens || !out_accept_len) return ERSD_EINVAL;
  if (N > 0) {
    if (!draft_logits) return ERSD_EINVAL;
    if (((uintptr_t)draft_logits & (elem_size(dt) - 1)) != 0) return ERSD_EALIGN;
  }
  TreeDesc tree;
  int D = 0, cmax = 1;
  st = build_tree(parent, N, &tree, &D, &cmax);
  if (st != ERSD_OK) return st;
  return verify_impl(target_logits, draft_logits, dt, tree, D, cmax, false, seeds, B, N + 1, N + 1,
                     V, T, out_tokens, out_accept_len, opts, cuda_stream);
}

int ersd_verify_noalloc(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                        const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                        int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream) {
  if (B < 1 || k < 0) return ERSD_EINVAL;
  if ((int64_t)B * ((int64_t)k + 1) > ERSD_NOALLOC_MAX_ROWS) return ERSD_ENOALLOC_LIMIT;
  ersd_opts o = read_opts(opts);
  if (o.workspace) return ERSD_EINVAL;  // this entry point brings its own scratch
  void* scratch = nullptr;
  const int st = noalloc_scratch(&scratch);
  if (st != ERSD_OK) return st;
  // The array keeps whatever the previous call left; the arrival counters (the first 16 bytes
  // of every slot this call uses) must start at zero.
  const cudaError_t e = cudaMemset2DAsync(scratch, sizeof(Slot), 0, 16, (size_t)B * ((size_t)k + 1),
                                          (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e);
  o.struct_size = sizeof o;
  o.workspace = scratch;
  o.workspace_bytes = kNoallocBytes;
  return ersd_verify(target_logits, draft_logits, dt, seeds, B, k, V, T, out_tokens, out_accept_len,
                     &o, cuda_stream);
}

int ersd_tree_depth(const int32_t* parent, int N) {
  if (!parent || N < 0 || N + 1 > ERSD_MAX_ROWS) return -1;
  TreeDesc tree;
  int D = 0, cmax = 1;
  if (build_tree(parent, N, &tree, &D, &cmax) != ERSD_OK) return -1;
  return D;
}

int ersd_row_keys(const void* row_logits, ersd_dtype dt, int V, float T, uint64_t seed,
                  uint32_t seq_id, uint32_t position, int mode, float* out_keys, void* cuda_stream) {
  if (!row_logits || !out_keys || V < 1 || !temp_ok(T) || (mode != 0 && mode != 1)) return ERSD_EINVAL;
  if (dt != ERSD_F32 && dt != ERSD_BF16) return ERSD_EINVAL;
  if (((uintptr_t)row_logits & (elem_size(dt) - 1)) != 0 || ((uintptr_t)out_keys & 3) != 0)
    return ERSD_EALIGN;
  const int threads = 256, blocks = (V + threads - 1) / threads;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (dt == ERSD_BF16)
    ersd_row_keys_kernel<ERSD_BF16><<<blocks, threads, 0, st>>>(row_logits, V, T, seed, seq_id, position, mode, out_keys);
  else
    ersd_row_keys_kernel<ERSD_F32><<<blocks, threads, 0, st>>>(row_logits, V, T, seed, seq_id, position, mode, out_keys);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

size_t ersd_workspace_bytes(int B, int rows_per_seq) {
  if (B < 1 || rows_per_seq < 1) return 0;
  return workspace_bytes(B, rows_per_seq);
}

int ersd_workspace_init(void* workspace, size_t bytes, void* cuda_stream) {
  if (!workspace) return ERSD_EINVAL;
  const cudaError_t e = cudaMemsetAsync(workspace, 0, bytes, (cudaStream_t)cuda_stream);
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

const char* ersd_status_string(int status) {
  switch (status) {
    case ERSD_OK: return "ok";
    case ERSD_EINVAL: return "invalid argument";
    case ERSD_EALIGN: return "misaligned pointer";
    case ERSD_EUNSUPPORTED: return "size beyond a compiled limit";
    case ERSD_ECUDA: return "CUDA runtime error";
    case ERSD_EWORKSPACE: return "workspace too small";
    case ERSD_ENOALLOC_LIMIT:
      return "B * (k + 1) exceeds ERSD_NOALLOC_MAX_ROWS, the capacity of ersd_verify_noalloc's built-in scratch";
    default: return "unknown status";
  }
}

int ersd_last_cuda_error(void) { return g_last_cuda_error; }

int ersd_version(void) { return 100; }

}  // extern "C"
