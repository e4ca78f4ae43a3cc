// libersd: exponential-race speculative decoding kernels for sm_100a and their C entry points.
//
// One thread block streams one chunk of one logit row (or of a draft/target
// row pair that shares its race variables).  Logits arrive through a
// shared-memory ring filled by cp.async; per group of eight vocabulary indices
// a thread draws the Philox words and compares one cheap lower bound of the
// eight race keys with the block's running threshold.  The few groups that
// survive are screened index by index in single precision and the survivors of
// that are decided in double precision and kept in per-warp sorted lists.
// Lists are merged per block, exchanged through a small workspace, and the
// last block of a sequence turns the winners into the accepted prefix
// (sequence scan or tree walk) in the same launch.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "ersd.h"
#include "ersd_math.cuh"

#ifndef ERSD_MIN_BLOCKS
#define ERSD_MIN_BLOCKS 4  // resident blocks per SM the register allocation aims for
#endif

namespace ersd {

#ifndef ERSD_THREADS
#define ERSD_THREADS 256
#endif
constexpr int kThreads = ERSD_THREADS;
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
  unsigned tau_code[2];  // per role: best threshold published so far (0 = none), see code_of_tau
  int pad;
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
  const int32_t* given_tok;  // [B, k] drafted tokens when they are given instead of draft rows
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

// 16-byte asynchronous copy global -> shared (bypasses L1); completion is tracked per thread.
__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gptr) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Geometry per logit type: a thread owns eight consecutive logits of a tile, i.e. kVec 16-byte
// vectors per role; the shared-memory ring holds kStages tiles per role (32 KB either way).
template <int DT>
struct Geo;
template <>
struct Geo<ERSD_BF16> {
  static constexpr int kVec = 1, kStages = 4;
};
template <>
struct Geo<ERSD_F32> {
  static constexpr int kVec = 2, kStages = 2;
};

template <int DT>
struct Raw {
  uint4 v[Geo<DT>::kVec];
};

// Eight logits starting at element i0 of a row; elements at or beyond `vend` read as NaN.
template <int DT>
__device__ __forceinline__ Raw<DT> fetch(const void* row, int i0, int vend, bool aligned) {
  Raw<DT> r;
  if constexpr (DT == ERSD_BF16) {
    const uint16_t* p = (const uint16_t*)row;
    if (aligned && i0 + kPerThread <= vend) {
      r.v[0] = ldg_stream(p + i0);
    } else {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int e0 = i0 + 2 * j, e1 = e0 + 1;
        const uint32_t lo = (e0 < vend) ? (uint32_t)__ldg(p + e0) : 0x7FC0u;
        const uint32_t hi = (e1 < vend) ? (uint32_t)__ldg(p + e1) : 0x7FC0u;
        w[j] = lo | (hi << 16);
      }
      r.v[0] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  } else {
    const uint32_t* p = (const uint32_t*)row;
    if (aligned && i0 + kPerThread <= vend) {
      r.v[0] = ldg_stream(p + i0);
      r.v[1] = ldg_stream(p + i0 + 4);
    } else {
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = (i0 + j < vend) ? __ldg(p + i0 + j) : 0x7FC00000u;
      r.v[0] = make_uint4(w[0], w[1], w[2], w[3]);
      r.v[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
  return r;
}

__device__ __forceinline__ void decode(const Raw<ERSD_BF16>& r, float z[8]) {
  const uint32_t w[4] = {r.v[0].x, r.v[0].y, r.v[0].z, r.v[0].w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    z[2 * j] = __uint_as_float(w[j] << 16);
    z[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void decode(const Raw<ERSD_F32>& r, float z[8]) {
  z[0] = __uint_as_float(r.v[0].x); z[1] = __uint_as_float(r.v[0].y);
  z[2] = __uint_as_float(r.v[0].z); z[3] = __uint_as_float(r.v[0].w);
  z[4] = __uint_as_float(r.v[1].x); z[5] = __uint_as_float(r.v[1].y);
  z[6] = __uint_as_float(r.v[1].z); z[7] = __uint_as_float(r.v[1].w);
}

// Logit j (0..7) of a thread's slice as staged in shared memory.
template <int DT>
__device__ __forceinline__ float staged_logit(const uint4* raw, int j) {
  if constexpr (DT == ERSD_BF16) return __uint_as_float((uint32_t)((const uint16_t*)raw)[j] << 16);
  else return ((const float*)raw)[j];
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
};

// Upper bound, in the screening keys' log2 units, of a double key in natural-log units.
__device__ __forceinline__ float tau_of_exact(double key) {
  const float t = (float)(key * 1.4426950408889634);
  return fmaf(fabsf(t), 2.384185791015625e-7f, t);
}

// Value a thread-tile's lower bound (which carries an offset of 32, see stream_tiles) is compared
// with: everything above it is out of the race for threshold tau.
__device__ __forceinline__ float lim_of_tau(float tau) {
  return fmaf(fabsf(tau), 9.5367431640625e-7f, tau) + 32.001953125f;
}

// Thresholds travel between the chunks of a row through the workspace as unsigned codes that
// grow as the threshold falls, with 0 (the workspace's resting state) meaning "none yet".
__device__ __forceinline__ unsigned code_of_tau(float tau) { return (unsigned)ord_of(-tau) ^ 0x80000000u; }
__device__ __forceinline__ float tau_of_code(unsigned code) {
  return code == 0u ? INFINITY : -float_of((int)(code ^ 0x80000000u));
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

// Shared-memory float minimum (rare path).
__device__ __forceinline__ void smem_min(float* addr, float v) {
  float old = *(volatile float*)addr;
  while (v < old) {
    const float seen = __int_as_float(atomicCAS((int*)addr, __float_as_int(old), __float_as_int(v)));
    if (seen == old) break;
    old = seen;
  }
}

// Upper bound of the eight logits of a thread's slice (NaN ignored; NaN if all are NaN).
__device__ __forceinline__ float logits_upper_bound(const Raw<ERSD_BF16>& r) {
  uint32_t m01, m23, m;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(m01) : "r"(r.v[0].x), "r"(r.v[0].y));
  asm("max.bf16x2 %0, %1, %2;" : "=r"(m23) : "r"(r.v[0].z), "r"(r.v[0].w));
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
  const float a = fmaxf(fmaxf(__uint_as_float(r.v[0].x), __uint_as_float(r.v[0].y)),
                        fmaxf(__uint_as_float(r.v[0].z), __uint_as_float(r.v[0].w)));
  const float b = fmaxf(fmaxf(__uint_as_float(r.v[1].x), __uint_as_float(r.v[1].y)),
                        fmaxf(__uint_as_float(r.v[1].z), __uint_as_float(r.v[1].w)));
  return fmaxf(a, b);
}

// ---------------------------------------------------------------------------------------------
// block state
// ---------------------------------------------------------------------------------------------
struct RoleInfo {
  const char* row;  // first element of the role's logit row
  int c;            // arrivals wanted
  int aligned;      // rows start on 16-byte boundaries
};

// What the block works on (written by thread 0 in setup_piece, read by everybody after it).
struct Job {
  int unit, b, r, s;   // logit row (b * rows + r), sequence, row in the sequence, chunk of the row
  int cq, c0;          // children of the row's node (0: no draft row), arrivals wanted from the target row
  int v0, v1;          // vocabulary range of the chunk
  int valid_T;
  float T, c2;         // temperature; keys are screened in log2 units: lg2(e) - z * c2
};

template <int DT>
struct __align__(16) Shared {
  // streaming ring: [stage][role][vector][thread], filled by cp.async, each thread reading back
  // only what it copied itself
  uint4 ring[Geo<DT>::kStages][2][Geo<DT>::kVec][kThreads];
  // per warp and role: the smallest (key, id) pairs seen so far, ascending
  Entry list[2][kWarps][ERSD_MAX_TOP_C];
  PhiloxRow philox;
  double inv_T;  // 1 / T of the row being raced (0 for greedy rows)
  RoleInfo role[2];
  float tau[2];  // log2 units: no index whose true key exceeds tau[r] can be among the first c
  alignas(8) float lim[2];  // lim_of_tau(tau[r])
  int last;
  Job job;
  int ttok[ERSD_MAX_ROWS], dtok[ERSD_MAX_ROWS];
  float tkey[ERSD_MAX_ROWS], dkey[ERSD_MAX_ROWS];
};

// The block's state lives at the start of dynamic shared memory; every function names it
// through this accessor, so the compiler sees shared-space addresses (no generic loads) and no
// pointer travels through the out-of-line calls.
extern __shared__ __align__(16) unsigned char ersd_dyn_smem[];
template <int DT>
__device__ __forceinline__ Shared<DT>& block_state() {
  return *reinterpret_cast<Shared<DT>*>(ersd_dyn_smem);
}

// After an insertion into warp `warp`'s list of role r: its c-th key bounds the role's threshold.
template <int DT>
__device__ __forceinline__ void publish_threshold(Shared<DT>& sh, int r, int warp, int lane) {
  const double kc = sh.list[r][warp][sh.role[r].c - 1].key;
  if (lane == 0 && kc < (double)INFINITY && kc > -(double)INFINITY) {
    const float tau = tau_of_exact(kc);
    smem_min(&sh.tau[r], tau);
    smem_min(&sh.lim[r], lim_of_tau(tau));
  }
}

// Logit j (0..7) of thread `t`'s slice of role `role` in ring stage `stage`.
template <int DT>
__device__ __forceinline__ float ring_logit(const Shared<DT>& sh, int stage, int role, int t, int j) {
  if constexpr (DT == ERSD_BF16) {
    return __uint_as_float((uint32_t)((const uint16_t*)&sh.ring[stage][role][0][t])[j] << 16);
  } else {
    return ((const float*)&sh.ring[stage][role][j >> 2][t])[j & 3];
  }
}

// The rare path of a tile.  Lanes whose `bits` are non-zero own eight indices (starting at their
// i0, logits in ring stage `stage`) that the cheap bound could not rule out for the roles named
// by the bits.  One such lane at a time is served by the warp: lanes 0-7 (role 0) and 8-15
// (role 1) each take one index, draw its Philox word again, form the accurate single-precision
// key and, if it is within the slack of the threshold, the double-precision key that decides;
// survivors enter the warp's list.
template <int DT>
__device__ __noinline__ void settle_tile(int stage, int i0, unsigned bits, float c2, float T) {
  Shared<DT>& sh = block_state<DT>();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool greedy = (T == 0.0f);
  __syncwarp();  // every lane's ring slot is complete and visible to the warp
  unsigned who = __ballot_sync(kFull, bits != 0);
  while (who) {
    const int src = __ffs(who) - 1;
    who &= who - 1;
    const int i0s = __shfl_sync(kFull, i0, src);
    const unsigned bs = __shfl_sync(kFull, bits, src);
    const int j = lane & 7, role = (lane >> 3) & 1;
    double dk = (double)INFINITY;
    if (lane < 16 && ((bs >> role) & 1u)) {
      uint32_t w[4];
      sh.philox.words(((uint32_t)i0s >> 2) + (uint32_t)(j >> 2), w);
      const uint32_t x = (j & 2) ? ((j & 1) ? w[3] : w[2]) : ((j & 1) ? w[1] : w[0]);
      const float z = ring_logit<DT>(sh, stage, role, warp * 32 + src, j);
      const float a = fmaf(-z, c2, greedy ? 0.0f : screen_lg2_e(x));
      const float tau = *(volatile float*)&sh.tau[role];
      if (a <= tau + screen_slack(tau)) dk = exact_key(x, z, sh.inv_T, greedy);
    }
    unsigned act = __ballot_sync(kFull, dk < (double)INFINITY);
    unsigned touched = 0;
    while (act) {
      const int s = __ffs(act) - 1;
      act &= act - 1;
      const double k = __shfl_sync(kFull, dk, s);
      const int r = s >> 3;
      Entry* L = sh.list[r][warp];
      WarpList wl;
      wl.key = L[lane].key;
      wl.idx = L[lane].idx;
      wl.insert(k, i0s + (s & 7), lane);
      L[lane].key = wl.key;
      L[lane].idx = wl.idx;
      touched |= 1u << r;
    }
    __syncwarp();
    if (touched & 1u) publish_threshold(sh, 0, warp, lane);
    if (touched & 2u) publish_threshold(sh, 1, warp, lane);
  }
  __syncwarp();  // nobody overwrites a ring slot that a lane is still reading
}

// A tile looked at index by index: the first tile of a piece when no threshold exists yet (the
// tile must yield one), a ragged last tile, and every tile of rows that are not 16-byte
// aligned.  Per role the c-th smallest of the lanes' best accurate single-precision keys, plus
// slack, is an upper bound of the c-th smallest true key; everything within the slack of the
// threshold goes to settle_tile, which finds the logits in ring stage `stage` (free at these
// moments: the streaming loop has no copy in flight into it).
template <int DT, int NR>
__device__ __noinline__ void edge_tile(int stage, int i0, int vend, float c2, float T) {
  Shared<DT>& sh = block_state<DT>();
  const int lane = threadIdx.x & 31;
  const bool greedy = (T == 0.0f);
  Raw<DT> raw[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) {
    raw[r] = fetch<DT>(sh.role[r].row, i0, vend, sh.role[r].aligned != 0);
#pragma unroll
    for (int v = 0; v < Geo<DT>::kVec; ++v) sh.ring[stage][r][v][threadIdx.x] = raw[r].v[v];
  }
  uint32_t xs[8];
  sh.philox.words((uint32_t)i0 >> 2, xs);
  sh.philox.words(((uint32_t)i0 >> 2) + 1u, xs + 4);
  float lg[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) lg[j] = greedy ? 0.0f : screen_lg2_e(xs[j]);
  unsigned bits = 0;
#pragma unroll
  for (int r = 0; r < NR; ++r) {
    float z[8];
    decode(raw[r], z);
    float m = INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) m = fminf(m, fmaf(-z[j], c2, lg[j]));
    const float tau_in = *(volatile float*)&sh.tau[r];
    const float theta = cth_smallest(m, sh.role[r].c, lane);
    const float tau = fminf(tau_in, theta + screen_slack(theta));
    if (lane == 0 && tau < tau_in) {
      smem_min(&sh.tau[r], tau);
      smem_min(&sh.lim[r], lim_of_tau(tau));
    }
    if (m <= tau + screen_slack(tau)) bits |= 1u << r;
  }
  __syncwarp();
  if (__any_sync(kFull, bits != 0)) settle_tile<DT>(stage, i0, bits, c2, T);
}

// The streaming loop over `ntiles` full tiles of 16-byte aligned rows; the thread's first index is
// i0.  Per thread and tile of eight indices: two Philox calls, the smallest of the eight words,
// the largest of the eight logits per role, and one comparison per role of
//     lg2(x_min) - z_max * c2      (a lower bound of all eight keys, shifted by 32:
//                                   lg2(e) >= lg2(w) > lg2(x) - 32)
// against the block's threshold.  Only when some lane of the warp cannot rule its eight indices
// out does the warp leave the loop body for settle_tile.  Logits reach the thread through a
// shared-memory ring that cp.async keeps kStages - 1 tiles ahead.
template <int DT, int NR>
struct Streamer {
  static constexpr int kVec = Geo<DT>::kVec, kStages = Geo<DT>::kStages;
  static constexpr int kElem = (DT == ERSD_BF16) ? 2 : 4;
  static constexpr uint32_t kStageBytes = 2 * kVec * kThreads * 16;
  const char* src[NR];  // next tile to request, this thread's slice
  int requested, ntiles;

  __device__ __forceinline__ void request_one(uint32_t ring0) {
    if (requested < ntiles) {
      const uint32_t base = ring0 + (uint32_t)(requested % kStages) * kStageBytes;
#pragma unroll
      for (int r = 0; r < NR; ++r) {
#pragma unroll
        for (int v = 0; v < kVec; ++v)
          cp_async16(base + (uint32_t)((r * kVec + v) * kThreads * 16), src[r] + v * 16);
        src[r] += (size_t)kTile * kElem;
      }
    }
    ++requested;
    cp_async_commit();
  }

  // Requests the first kStages - 1 tiles; call before any other work so the copies overlap it.
  __device__ __forceinline__ void begin(const char* const* rows, int i0, int ntiles_) {
    Shared<DT>* sh = &block_state<DT>();
    ntiles = ntiles_;
    requested = 0;
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(&sh->ring[0][0][0][threadIdx.x]);
#pragma unroll
    for (int r = 0; r < NR; ++r) src[r] = rows[r] + (size_t)i0 * kElem;
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) request_one(ring0);
  }

  __device__ __forceinline__ void run(int i0, float c2, float T) {
    Shared<DT>* sh = &block_state<DT>();
    const bool greedy = (T == 0.0f);
    const PhiloxRow pr = sh->philox;
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(&sh->ring[0][0][0][threadIdx.x]);
    const uint32_t lim_addr = (uint32_t)__cvta_generic_to_shared(sh->lim);
    int t = 0;
    while (t < ntiles) {
      // inner loop: no call inside, left only when some lane cannot rule its indices out
      unsigned bits = 0;
      int stage = 0;
      for (; t < ntiles; ++t, i0 += kTile) {
        request_one(ring0);
        cp_async_wait<kStages - 1>();
        stage = t % kStages;
        float zub[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          Raw<DT> cur;
#pragma unroll
          for (int v = 0; v < kVec; ++v) cur.v[v] = sh->ring[stage][r][v][threadIdx.x];
          zub[r] = logits_upper_bound(cur);
        }
        uint32_t xs[8];
        pr.words((uint32_t)i0 >> 2, xs);
        pr.words(((uint32_t)i0 >> 2) + 1u, xs + 4);
        const uint32_t xm = min(__vimin3_u32(xs[0], xs[1], xs[2]),
                                __vimin3_u32(__vimin3_u32(xs[3], xs[4], xs[5]), xs[6], xs[7]));
        const float lgm = greedy ? 32.0f : lg2_fast((float)xm);
        float2 lim;  // both roles' comparison values in one volatile load
        asm volatile("ld.volatile.shared.v2.f32 {%0,%1}, [%2];" : "=f"(lim.x), "=f"(lim.y) : "r"(lim_addr));
        bits = 0;
        if (!(fmaf(-zub[0], c2, lgm) > lim.x)) bits |= 1u;
        if (NR == 2) {
          if (!(fmaf(-zub[NR - 1], c2, lgm) > lim.y)) bits |= 2u;
        }
        if (__any_sync(kFull, bits != 0)) break;
      }
      if (t < ntiles) {
        settle_tile<DT>(stage, i0, bits, c2, T);
        ++t;
        i0 += kTile;
      }
    }
  }
};

// The first tile of a chunk that starts with a threshold for every role: the same cheap test as
// in the streaming loop, on logits fetched with plain loads (and parked in ring stage `stage`
// for settle_tile).
template <int DT, int NR>
__device__ __noinline__ void first_tile(int stage, int i0, int vend, float c2, float T) {
  Shared<DT>& sh = block_state<DT>();
  const bool greedy = (T == 0.0f);
  float zub[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) {
    const Raw<DT> raw = fetch<DT>(sh.role[r].row, i0, vend, true);
#pragma unroll
    for (int v = 0; v < Geo<DT>::kVec; ++v) sh.ring[stage][r][v][threadIdx.x] = raw.v[v];
    zub[r] = logits_upper_bound(raw);
  }
  uint32_t xs[8];
  sh.philox.words((uint32_t)i0 >> 2, xs);
  sh.philox.words(((uint32_t)i0 >> 2) + 1u, xs + 4);
  const uint32_t xm = min(__vimin3_u32(xs[0], xs[1], xs[2]),
                          __vimin3_u32(__vimin3_u32(xs[3], xs[4], xs[5]), xs[6], xs[7]));
  const float lgm = greedy ? 32.0f : lg2_fast((float)xm);
  unsigned bits = 0;
#pragma unroll
  for (int r = 0; r < NR; ++r)
    if (fmaf(-zub[r], c2, lgm) <= *(volatile float*)&sh.lim[r]) bits |= 1u << r;
  if (__any_sync(kFull, bits != 0)) settle_tile<DT>(stage, i0, bits, c2, T);
}

// One piece = chunk [v0, v1) of a logit row (NR = 1) or of a draft/target pair (NR = 2); rows[]
// point at the rows' first elements.  The streaming loop takes the full tiles after the first;
// the first tile yields the first threshold unless an earlier chunk of the row handed one down;
// a ragged last tile gets the cheap test with bounds-checked loads.
// (Inlined into the kernel, whose other parts are out-of-line calls: the loop then gets a
// register allocation of its own.)
template <int DT, int NR>
__device__ __forceinline__ void stream_piece(const char* const* rows, bool ring_ok, int v0, int v1,
                                             float c2, float T) {
  constexpr int kStages = Geo<DT>::kStages;
  Shared<DT>* sh = &block_state<DT>();
  const int tid = threadIdx.x;
  const int ntiles = (int)((unsigned)(v1 - v0 + kTile - 1) / kTile);
  const int nfull = (int)((unsigned)(v1 - v0) / kTile);  // tiles that lie fully inside the piece
  int i0 = v0 + tid * kPerThread;
  if (ring_ok) {
    Streamer<DT, NR> st;
    st.begin(rows, i0 + kTile, nfull > 1 ? nfull - 1 : 0);
    // (the requests above leave the last ring stage free for the first tile's logits)
    bool have_tau = (nfull >= 1);
#pragma unroll
    for (int r = 0; r < NR; ++r) have_tau = have_tau && (sh->tau[r] < INFINITY);
    if (have_tau) first_tile<DT, NR>(kStages - 1, i0, v1, c2, T);
    else edge_tile<DT, NR>(kStages - 1, i0, v1, c2, T);
    if (nfull > 1) st.run(i0 + kTile, c2, T);
    cp_async_wait<0>();
    if (ntiles > nfull && ntiles > 1) {
      // ragged last tile: the cheap test again (indices beyond the row read as NaN and never
      // pass) unless the chunk still has no threshold
      bool tau_now = true;
#pragma unroll
      for (int r = 0; r < NR; ++r) tau_now = tau_now && (*(volatile float*)&sh->tau[r] < INFINITY);
      if (tau_now) first_tile<DT, NR>(0, i0 + (ntiles - 1) * kTile, v1, c2, T);
      else edge_tile<DT, NR>(0, i0 + (ntiles - 1) * kTile, v1, c2, T);
    }
  } else {
    for (int t = 0; t < ntiles; ++t, i0 += kTile) edge_tile<DT, NR>(0, i0, v1, c2, T);
  }
}

// Merge `n` sorted partial lists of `c` entries each (global memory written by other blocks,
// n * c <= 64) into a fresh warp list.  All entries are fetched at once, two per lane, so the
// merge pays one memory round trip, not one per entry.
__device__ __forceinline__ void merge_partials(WarpList& L, const Entry* part, int n, int c,
                                               int lane) {
  const int total = n * c;
  double k0 = (double)INFINITY, k1 = (double)INFINITY;
  int i0 = 0x7FFFFFFF, i1 = 0x7FFFFFFF;  // unused slots carry idx = INT_MAX
  if (lane < total) {
    k0 = __ldcg(&part[lane].key);
    i0 = __ldcg(&part[lane].idx);
  }
  if (lane + 32 < total) {
    k1 = __ldcg(&part[lane + 32].key);
    i1 = __ldcg(&part[lane + 32].idx);
  }
  L.init();
  if (c == 1) {  // winners only: the smallest (key, idx) by a shuffle tree, result in lane 0
    if (k1 < k0 || (k1 == k0 && i1 < i0)) {
      k0 = k1;
      i0 = i1;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const double ok = __shfl_down_sync(kFull, k0, off);
      const int oi = __shfl_down_sync(kFull, i0, off);
      if (ok < k0 || (ok == k0 && oi < i0)) {
        k0 = ok;
        i0 = oi;
      }
    }
    if (lane == 0) {
      L.key = k0;
      L.idx = i0;
    }
    return;
  }
  for (int e = 0; e < total; ++e) {
    const double k = __shfl_sync(kFull, e < 32 ? k0 : k1, e & 31);
    const int i = __shfl_sync(kFull, e < 32 ? i0 : i1, e & 31);
    if (i != 0x7FFFFFFF) L.insert(k, i, lane);
  }
}

// Decodes the block's work item and prepares the shared state.  Work items are ordered
// chunk-major: every row's first chunk is scheduled before any second chunk, so that later
// chunks of a row usually start with the threshold an earlier one left in the workspace;
// within a chunk index rows follow tree.order (the heavier paired rows first).
template <int DT>
__device__ __noinline__ void setup_piece(const Params& p, const TreeDesc& tree) {
  Shared<DT>& sh = block_state<DT>();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // every thread decodes (cheap, no memory); single lanes of different warps then fill in the
  // parts of the state side by side, so that their memory latencies overlap
  const int s = blockIdx.z, ri = blockIdx.y, b = blockIdx.x;  // (no division: keeps these uniform)
  const int r = (p.mode == kSample) ? ri : (int)tree.order[ri];
  const int unit = b * p.rows + r;
  const int cq = (p.mode == kSample) ? 0 : (int)tree.nchild[r];
  const int c0 = (p.mode == kSample) ? p.c_sample : 1;
  if (lane == 0) {
    if (warp == 0) {
      const uint64_t seed = p.seeds[b];
      const uint32_t seq = p.seq_ids ? p.seq_ids[b] : (uint32_t)b;
      const uint32_t pos = (p.pos_offsets ? p.pos_offsets[b] : 0u) + (uint32_t)r;
      sh.philox.init(seed, seq, pos);
    } else if (warp == 1) {
      const float T = p.temps ? p.temps[(int64_t)b * p.ts_b + (int64_t)r * p.ts_r] : p.T;
      Job j;
      j.unit = unit; j.b = b; j.r = r; j.s = s; j.cq = cq; j.c0 = c0;
      j.v0 = s * p.per_chunk;
      j.v1 = min(p.V, j.v0 + p.per_chunk);
      j.valid_T = (T >= 0.0f && T < INFINITY);
      j.T = T;
      j.c2 = (T == 0.0f) ? kLog2e : (float)(1.4426950408889634 / (double)T);  // greedy: -z log2(e)
      sh.job = j;
      sh.inv_T = (T == 0.0f) ? 0.0 : 1.0 / (double)T;
    } else if (warp == 2) {
      const size_t es = (DT == ERSD_BF16) ? 2 : 4;
      sh.role[0].row = (const char*)p.target + (size_t)unit * (size_t)p.ld_t * es;
      sh.role[0].c = c0;
      sh.role[0].aligned = p.aligned_t;
      sh.role[1].row = cq > 0 ? (const char*)p.draft + ((size_t)b * p.draft_rows + r) * (size_t)p.ld_d * es
                              : nullptr;
      sh.role[1].c = cq > 0 ? cq : 1;
      sh.role[1].aligned = p.aligned_d;
    }
  }
  if (warp == 3 && lane < 2) {
    // thresholds handed down by earlier chunks of this row (any of them is a valid bound)
    const int q = lane;
    const float tau = (p.S > 1) ? tau_of_code(__ldcg(&p.slots[unit].tau_code[q])) : INFINITY;
    sh.tau[q] = tau;
    sh.lim[q] = (tau < INFINITY) ? lim_of_tau(tau) : INFINITY;
  }
  Entry e;
  e.key = (double)INFINITY;
  e.idx = 0x7FFFFFFF;
  e.pad = 0;
  sh.list[0][warp][lane] = e;
  sh.list[1][warp][lane] = e;
  __syncthreads();
}

// After the streaming: merges the warps' lists, hands the chunk's arrivals to the workspace and,
// in the block that completes the group (row in sample mode, sequence otherwise), turns the
// winners into the call's outputs.
template <int DT>
__device__ __noinline__ void finish_piece(const Params& p, const TreeDesc& tree) {
  Shared<DT>& sh = block_state<DT>();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = sh.job.unit, b = sh.job.b, s = sh.job.s, cq = sh.job.cq, c0 = sh.job.c0;
  // ---- block merge: warp `role` merges the eight warps' lists of that role ----
  const int nroles = cq > 0 ? 2 : 1;
  const bool direct = (p.mode == kSample && p.S == 1);
  if (warp < nroles) {
    const int role = warp;
    const int c = sh.role[role].c;
    WarpList L;
    if (c == 1) {  // winners only: lane w takes warp w's best, a shuffle tree finds the smallest
      L.key = lane < kWarps ? sh.list[role][lane][0].key : (double)INFINITY;
      L.idx = lane < kWarps ? sh.list[role][lane][0].idx : 0x7FFFFFFF;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const double ok = __shfl_down_sync(kFull, L.key, off);
        const int oi = __shfl_down_sync(kFull, L.idx, off);
        if (ok < L.key || (ok == L.key && oi < L.idx)) {
          L.key = ok;
          L.idx = oi;
        }
      }
    } else {
      L.key = sh.list[role][0][lane].key;
      L.idx = sh.list[role][0][lane].idx;
      for (int w = 1; w < kWarps; ++w) {
        for (int e = 0; e < c; ++e) {
          const Entry en = sh.list[role][w][e];
          if (en.idx == 0x7FFFFFFF) break;
          L.insert(en.key, en.idx, lane);
        }
      }
    }
    if (direct) {
      if (lane < c) {
        const bool ok = L.idx != 0x7FFFFFFF;
        const size_t o = (size_t)unit * c + lane;
        p.out_tokens[o] = ok ? L.idx : -1;
        if (p.out_key) p.out_key[o] = ok ? (float)L.key : INFINITY;
      }
    } else {
      if (lane < c) {
        Entry e;
        e.key = L.key;
        e.idx = L.idx;
        e.pad = 0;
        p.slots[unit].part[role][s * c + lane] = e;
      }
      // hand the threshold down to the row's later chunks
      const float tau = sh.tau[role];
      if (lane == 0 && tau < INFINITY) atomicMax(&p.slots[unit].tau_code[role], code_of_tau(tau));
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
    sh.last = (old == group_items - 1);
  }
  __syncthreads();
  if (!sh.last) return;
  __threadfence();
  // leave the workspace ready for the next call
  if (tid == 0) *counter = 0;
  if (p.mode == kSample) {
    if (tid < 2) p.slots[unit].tau_code[tid] = 0u;
  } else {
    for (int n = tid; n < p.rows * 2; n += kThreads) p.slots[b * p.rows + (n >> 1)].tau_code[n & 1] = 0u;
  }

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
        sh.ttok[n] = ok ? L.idx : -1;
        sh.tkey[n] = ok ? (float)L.key : INFINITY;
      }
    } else if (lane < c) {
      int m = tree.first_child[n];  // the child of rank `lane`
      for (int q = 0; q < lane; ++q) m = tree.next_sib[m];
      sh.dtok[m] = ok ? L.idx : -1;
      sh.dkey[m] = ok ? (float)L.key : INFINITY;
    }
  }
  if (p.given_tok) {  // drafted earlier: node n holds the token drafted at position n - 1
    for (int n = 1 + tid; n < p.rows; n += kThreads) {
      sh.dtok[n] = p.given_tok[(size_t)b * (p.rows - 1) + (n - 1)];
      sh.dkey[n] = INFINITY;
    }
  }
  if (tid == 0) {
    sh.dtok[0] = -1;
    sh.dkey[0] = INFINITY;
  }
  __syncthreads();

  const int cols = p.depth + 1;
  for (int d = tid; d < cols; d += kThreads) {
    p.out_tokens[(size_t)b * cols + d] = -1;
    if (p.out_path) p.out_path[(size_t)b * cols + d] = -1;
  }
  for (int n = tid; n < p.rows; n += kThreads) {
    const size_t o = (size_t)b * p.rows + n;
    if (p.out_target_tok) p.out_target_tok[o] = sh.ttok[n];
    if (p.out_target_key) p.out_target_key[o] = sh.tkey[n];
    if (p.chain_outputs) {
      if (n >= 1) {
        const size_t od = (size_t)b * (p.rows - 1) + (n - 1);
        if (p.out_draft_tok) p.out_draft_tok[od] = sh.dtok[n];
        if (p.out_draft_key) p.out_draft_key[od] = sh.dkey[n];
      }
    } else {
      if (p.out_draft_tok) p.out_draft_tok[o] = sh.dtok[n];
      if (p.out_draft_key) p.out_draft_key[o] = sh.dkey[n];
    }
  }
  __syncthreads();
  if (tid == 0) {
    // Walk down from the root while the target winner of the current node's race is the
    // token drafted at one of its children.
    int cur = 0, depth = 0;
    for (;;) {
      const int w = sh.ttok[cur];
      p.out_tokens[(size_t)b * cols + depth] = w;
      if (p.out_path) p.out_path[(size_t)b * cols + depth] = cur;
      int next = -1;
      if (w >= 0) {
        for (int m = tree.first_child[cur]; m >= 0; m = tree.next_sib[m]) {
          if (sh.dtok[m] == w) {
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
__global__ void __launch_bounds__(kThreads, ERSD_MIN_BLOCKS)
ersd_race_kernel(const __grid_constant__ Params p, const __grid_constant__ TreeDesc tree) {
  // The same decode as in setup_piece, from launch parameters only: everything here is uniform
  // over the block, and the compiler can tell.
  const int s = blockIdx.z, ri = blockIdx.y, b = blockIdx.x;  // (no division: keeps these uniform)
  const int r = (p.mode == kSample) ? ri : (int)tree.order[ri];
  const int cq = (p.mode == kSample) ? 0 : (int)tree.nchild[r];
  const int v0 = s * p.per_chunk;
  const int v1 = min(p.V, v0 + p.per_chunk);
  const size_t es = (DT == ERSD_BF16) ? 2 : 4;
  const char* rows[2];
  rows[0] = (const char*)p.target + ((size_t)b * p.rows + r) * (size_t)p.ld_t * es;
  rows[1] = (const char*)p.draft + ((size_t)b * p.draft_rows + r) * (size_t)p.ld_d * es;
  const bool ring_ok = p.aligned_t && (cq == 0 || p.aligned_d);

  setup_piece<DT>(p, tree);
  {
    const Job& j = block_state<DT>().job;
    if (j.valid_T) {  // a row with an invalid temperature has no arrivals
      if (cq > 0) stream_piece<DT, 2>(rows, ring_ok, v0, v1, j.c2, j.T);
      else stream_piece<DT, 1>(rows, ring_ok, v0, v1, j.c2, j.T);
    }
  }
  __syncthreads();
  finish_piece<DT>(p, tree);
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
  } else if (mode == 2) {
    // the deciding key against the CUDA math library's log / log1p, in units of 1e-12
    const double w = ((double)x + 0.5) * (1.0 / 4294967296.0);
    const double ref = (T == 0.0f) ? -(double)z : log(-log1p(-w)) - (double)z / (double)T;
    out[i] = (float)((exact_key(x, z, T) - ref) * 1e12);
  } else {
    const float c2 = (float)(1.4426950408889634 / (T == 0.0f ? 1.0 : (double)T));
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

#ifndef ERSD_MIN_CHUNK_TILES
#define ERSD_MIN_CHUNK_TILES 8  // smallest chunk of a row that the default split makes
#endif

// Thread blocks per row.  At least one work item per resident-block slot, and two chunks per
// row when rows are long: the hardware's block scheduler then evens out rows of different cost
// and the last wave is made of half rows.  More chunks do not pay: each costs a block about as
// much set-up, barrier and merge time as eight tiles of streaming (measured).
static int choose_split(const ersd_opts& o, int64_t units, int V, int cmax) {
  int smax = kPartCap / cmax;
  if (smax > ERSD_MAX_SPLIT) smax = ERSD_MAX_SPLIT;
  if (smax < 1) smax = 1;
  const int ntiles = (V + kTile - 1) / kTile;
  int S;
  if (o.split_v) {
    S = (int)o.split_v;
    if (S > ntiles) S = ntiles;
  } else {
    const int64_t slots = 148 * ERSD_MIN_BLOCKS;
    S = (int)((slots + units - 1) / units);
    if (S < 2 && ntiles >= 4 * ERSD_MIN_CHUNK_TILES) S = 2;
    const int by_v = ntiles / ERSD_MIN_CHUNK_TILES;
    if (S > by_v) S = by_v;
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

// Four resident blocks per SM need about 180 KB of shared memory: ask for the largest carveout
// (a hint to the driver; set once per device and kernel).
static int prefer_shared_memory() {
  static std::mutex m;
  static bool done[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return ERSD_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(m);
  if (!done[dev]) {
    e = cudaFuncSetAttribute(ersd_race_kernel<ERSD_BF16>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(ersd_race_kernel<ERSD_F32>, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(ersd_race_kernel<ERSD_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)sizeof(Shared<ERSD_BF16>));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(ersd_race_kernel<ERSD_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)sizeof(Shared<ERSD_F32>));
    if (e != cudaSuccess) return cuda_fail(e);
    done[dev] = true;
  }
  return ERSD_OK;
}

static int launch(const Params& p, const TreeDesc& tree, int dt, cudaStream_t st) {
  // grid (sequence, row in launch order, chunk): blocks are dispatched x fastest, z slowest, which
  // is the chunk-major order the kernel counts on, and the kernel needs no division to decode
  if (p.rows > 65535 || p.S > 65535) return ERSD_EUNSUPPORTED;
  const dim3 grid((unsigned)p.B, (unsigned)p.rows, (unsigned)p.S);
  const int pst = prefer_shared_memory();
  if (pst != ERSD_OK) return pst;
  if (dt == ERSD_BF16) ersd_race_kernel<ERSD_BF16><<<grid, kThreads, sizeof(Shared<ERSD_BF16>), st>>>(p, tree);
  else ersd_race_kernel<ERSD_F32><<<grid, kThreads, sizeof(Shared<ERSD_F32>), st>>>(p, tree);
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
                       const ersd_opts* opts, void* stream, const int32_t* given_tok = nullptr) {
  const ersd_opts o = read_opts(opts);
  Params p;
  memset(&p, 0, sizeof p);
  fill_common(p, o, seeds, B, rows, V, T);
  p.target = target;
  p.draft = draft;
  p.given_tok = given_tok;
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

int ersd_verify_tokens(const void* target_logits, const int32_t* draft_tokens, ersd_dtype dt,
                       const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                       int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream) {
  if (k < 0) return ERSD_EINVAL;
  if (k + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  int st = check_common(target_logits, dt, seeds, B, k + 1, V, T);
  if (st != ERSD_OK) return st;
  if (!out_tokens || !out_accept_len) return ERSD_EINVAL;
  if (k > 0) {
    if (!draft_tokens) return ERSD_EINVAL;
    if (((uintptr_t)draft_tokens & 3) != 0) return ERSD_EALIGN;
  }
  int32_t parent[ERSD_MAX_ROWS];
  for (int n = 0; n <= k; ++n) parent[n] = n - 1;
  TreeDesc tree;
  int D = 0, cmax = 1;
  st = build_tree(parent, k, &tree, &D, &cmax);
  if (st != ERSD_OK) return st;
  // the chain keeps its shape for the walk, but no row has a draft row to race
  for (int n = 0; n <= k; ++n) {
    tree.nchild[n] = 0;
    tree.order[n] = (uint8_t)n;
  }
  return verify_impl(target_logits, nullptr, dt, tree, D, 1, true, seeds, B, k + 1, k, V, T, out_tokens,
                     out_accept_len, opts, cuda_stream, k > 0 ? draft_tokens : nullptr);
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
  if (!row_logits || !out_keys || V < 1 || !temp_ok(T) || (mode < 0 || mode > 2)) return ERSD_EINVAL;
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

int ersd_version(void) { return 102; }

}  // extern "C"
