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
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "ersd.h"
#include "ersd_math.cuh"

namespace ersd {

constexpr int kPerThread = 8;  // consecutive vocabulary indices a thread owns in a tile
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
  int threads;  // threads per block of the kernel variant this call launches (128 or 256)
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
  uint32_t* near_tie;    // count of races with two consecutive arrivals closer than 1e-5 (nullable)
  int extra;             // 1 when near-ties are counted: every race is run for one more arrival
  int top_cmax;          // cluster kernel for several arrivals: most arrivals any race of the call wants
  int top_split;         // the same kernel: 0, or 1 + the number of nodes with children when every row gets its own cluster
  Slot* slots;
};

// ---------------------------------------------------------------------------------------------
// The kernel, compiled for two block sizes: many rows are raced by 128-thread blocks (seven per
// SM: more, smaller work items and a shorter last wave), few rows by 256-thread blocks (four per
// SM: a row's thresholds are shared by more warps, half as many blocks to set up).
// ---------------------------------------------------------------------------------------------
namespace b256 {
constexpr int kThreads = 256, kMinBlocks = 4;
constexpr bool kMany = false;
#include "ersd_kernel.inc"
}  // namespace b256
namespace b128 {
constexpr int kThreads = 128, kMinBlocks = 7;
constexpr bool kMany = false;
#include "ersd_kernel.inc"
}  // namespace b128
// The same two for calls of few rows with races that want several arrivals (tree and batch
// drafting, top_c > 1) and for every call with a race of more than 32 arrivals: see launch().
namespace b256m {
constexpr int kThreads = 256, kMinBlocks = 4;
constexpr bool kMany = true;
#include "ersd_kernel.inc"
}  // namespace b256m
namespace b128m {
constexpr int kThreads = 128, kMinBlocks = 7;
constexpr bool kMany = true;
#include "ersd_kernel.inc"
}  // namespace b128m
namespace b256 {
#include "ersd_cluster.inc"
#include "ersd_cluster_top.inc"
}  // namespace b256

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
static thread_local char g_last_launch[160] = "";  // ersd_last_launch(): what this thread's last call launched

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

// The private workspace of a device is zeroed on the stream of the call that (re)allocates it, so
// that the zeroing is ordered before that call's kernel whatever kind of stream it is.
static int get_workspace(const ersd_opts& o, size_t need, void** ws, cudaStream_t stream) {
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
    e = cudaMemsetAsync(w.ptr, 0, grow, stream);
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

constexpr int kMinChunkTiles = 8;  // smallest chunk of a row that the default split makes

// Multiprocessors of the current device (asked once per device; 148 on a B200).
static int sm_count() {
  static std::mutex m;
  static int count[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  std::lock_guard<std::mutex> lock(m);
  if (!count[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      n = 148;
    }
    count[dev] = n;
  }
  return count[dev];
}

// Block size of a call: opts->block_threads if given, else 128-thread blocks when there are enough
// rows to give every one of their (twice as many) resident-block slots a chunk, 256 otherwise.
static int choose_threads(const ersd_opts& o, int64_t units, int* threads) {
  if (o.block_threads == 0) *threads = units >= (int64_t)sm_count() * b128::kMinBlocks ? 128 : 256;
  else if (o.block_threads == 128 || o.block_threads == 256) *threads = (int)o.block_threads;
  else return ERSD_EINVAL;
  return ERSD_OK;
}

// Thread blocks per row.
static int choose_split(const ersd_opts& o, int64_t units, int V, int cmax, int threads) {
  int smax = kPartCap / cmax;
  if (smax > ERSD_MAX_SPLIT) smax = ERSD_MAX_SPLIT;
  if (smax < 1) smax = 1;
  const int tile = threads * kPerThread;
  const int ntiles = (V + tile - 1) / tile;
  int S;
  if (o.split_v) {
    S = (int)o.split_v;
    if (S > ntiles) S = ntiles;
  } else {
    // about 1.7 blocks per SM: a block costs as much set-up, first threshold, merge and finish as
    // eight tiles of streaming, so more chunks than the SMs need to be busy only add work
    // (measured on calls of 48 to 400 rows: 5 to 15 % quicker than one block per resident slot)
    const int64_t slots = (int64_t)sm_count() * (threads == 128 ? b128::kMinBlocks : b256::kMinBlocks);
    // (races of several arrivals: their rare path is the long one, and shorter chunks bound it;
    // there a block per resident slot stays the better choice)
    const int64_t wanted = cmax > 1 ? slots : ((int64_t)sm_count() * 27) / 16;
    S = (int)((wanted + units - 1) / units);
    // whole rows that make more than one wave, and rows of uneven cost (trees): halves even out the last wave
    if (S < 2 && (units > slots || cmax > 1) && (int64_t)ntiles * tile >= 4 * kMinChunkTiles * b256::kTile) S = 2;
    const int by_v = ntiles / kMinChunkTiles;
    if (S > by_v) S = by_v;
  }
  if (S > smax) S = smax;
  if (S < 1) S = 1;
  return S;
}

static void set_chunks(Params& p, int S) {
  const int tile = p.threads * kPerThread;
  int per = (p.V + S - 1) / S;
  per = (per + tile - 1) / tile * tile;
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
    e = cudaSuccess;
    const void* kernels[8] = {(const void*)b256::ersd_race_kernel<ERSD_BF16>, (const void*)b256::ersd_race_kernel<ERSD_F32>,
                              (const void*)b128::ersd_race_kernel<ERSD_BF16>, (const void*)b128::ersd_race_kernel<ERSD_F32>,
                              (const void*)b256m::ersd_race_kernel<ERSD_BF16>, (const void*)b256m::ersd_race_kernel<ERSD_F32>,
                              (const void*)b128m::ersd_race_kernel<ERSD_BF16>, (const void*)b128m::ersd_race_kernel<ERSD_F32>};
    const int smem[8] = {(int)sizeof(b256::Shared<ERSD_BF16>), (int)sizeof(b256::Shared<ERSD_F32>),
                         (int)sizeof(b128::Shared<ERSD_BF16>), (int)sizeof(b128::Shared<ERSD_F32>),
                         (int)sizeof(b256m::Shared<ERSD_BF16>), (int)sizeof(b256m::Shared<ERSD_F32>),
                         (int)sizeof(b128m::Shared<ERSD_BF16>), (int)sizeof(b128m::Shared<ERSD_F32>)};
    for (int q = 0; q < 8 && e == cudaSuccess; ++q) {
      e = cudaFuncSetAttribute(kernels[q], cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(kernels[q], cudaFuncAttributeMaxDynamicSharedMemorySize, smem[q]);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    done[dev] = true;
  }
  return ERSD_OK;
}

// `many`: some race of the call wants several arrivals (a tree node with several children,
// top_c > 1).  Calls of up to two rows per SM then take the variant of the kernel that pools the
// block's decided indices (measured: a star of 8 at B=1 48 -> 42 us, the 17-node tree 35 -> 33 us;
// at 544 rows the pooling costs 0.7 % instead).
// cmax: most arrivals any race of the call wants.  The builds for races of several arrivals take
// calls of few rows (their loop is slower, their rare path quicker) and every call with a race of
// more than 32 arrivals (only they hold two list entries per lane).
static int launch(const Params& p, const TreeDesc& tree, int dt, int cmax, cudaStream_t st) {
  const bool many = cmax > 32 || (cmax > 1 && (int64_t)p.B * p.rows <= 2 * sm_count());
  // grid (sequence, row in launch order, chunk): blocks are dispatched x fastest, z slowest, which
  // is the chunk-major order the kernel counts on, and the kernel needs no division to decode
  if (p.rows > 65535 || p.S > 65535) return ERSD_EUNSUPPORTED;
  const dim3 grid((unsigned)p.B, (unsigned)p.rows, (unsigned)p.S);
  const int pst = prefer_shared_memory();
  if (pst != ERSD_OK) return pst;
  snprintf(g_last_launch, sizeof g_last_launch, "ersd_race_kernel<%s>%s: %d threads x (%d, %d, %d) blocks, %d chunk(s) per row",
           dt == ERSD_BF16 ? "bf16" : "f32", many ? " (pooled thresholds)" : "", p.threads, p.B, p.rows, p.S, p.S);
  if (many) {
    if (p.threads == 128) {
      if (dt == ERSD_BF16)
        b128m::ersd_race_kernel<ERSD_BF16><<<grid, 128, sizeof(b128m::Shared<ERSD_BF16>), st>>>(p, tree);
      else
        b128m::ersd_race_kernel<ERSD_F32><<<grid, 128, sizeof(b128m::Shared<ERSD_F32>), st>>>(p, tree);
    } else {
      if (dt == ERSD_BF16)
        b256m::ersd_race_kernel<ERSD_BF16><<<grid, 256, sizeof(b256m::Shared<ERSD_BF16>), st>>>(p, tree);
      else
        b256m::ersd_race_kernel<ERSD_F32><<<grid, 256, sizeof(b256m::Shared<ERSD_F32>), st>>>(p, tree);
    }
  } else if (p.threads == 128) {
    if (dt == ERSD_BF16)
      b128::ersd_race_kernel<ERSD_BF16><<<grid, 128, sizeof(b128::Shared<ERSD_BF16>), st>>>(p, tree);
    else
      b128::ersd_race_kernel<ERSD_F32><<<grid, 128, sizeof(b128::Shared<ERSD_F32>), st>>>(p, tree);
  } else {
    if (dt == ERSD_BF16)
      b256::ersd_race_kernel<ERSD_BF16><<<grid, 256, sizeof(b256::Shared<ERSD_BF16>), st>>>(p, tree);
    else
      b256::ersd_race_kernel<ERSD_F32><<<grid, 256, sizeof(b256::Shared<ERSD_F32>), st>>>(p, tree);
  }
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

// ---------------------------------------------------------------------------------------------
// Latency path of calls of few rows: one cluster of thread blocks per position (ersd_cluster.inc).
// ---------------------------------------------------------------------------------------------
// Default choice: the cluster kernel is taken while its blocks number up to 1280 (sampling: 160
// rows of 128256 logits) or, in verification (two rows per position), while the positions would
// make up to 704 blocks in clusters of full size (44 positions of 128256 logits); beyond that the
// streaming kernel's throughput wins (measured at V = 128256 and 32000).
constexpr int64_t kClusterAutoBlocksSample = 1280, kClusterAutoBlocksVerify = 704;
// The same for races of several arrivals (ersd_cluster_top.inc; three blocks per SM).
constexpr int64_t kClusterAutoBlocksTop = 600;
// ... and the number of blocks up to which a tree's rows get a cluster each (one block per SM and a half)
constexpr int64_t kClusterSplitBlocks = 384;
constexpr size_t kClusterSmemBytes = 200 * 1024;  // dynamic shared memory a block of the cluster kernels may use

// Tiles per block that fit (roles = rows raced together: 1, or 2 for a draft/target pair; cmax > 1:
// the kernel for races of several arrivals, which keeps its lists behind the rows).
static int cluster_max_tiles(int dt, int roles, int cmax) {
  const size_t per_tile = dt == ERSD_BF16 ? b256::cluster_role_bytes<ERSD_BF16>(1) : b256::cluster_role_bytes<ERSD_F32>(1);
  const size_t lists = cmax > 1 ? b256::top_list_bytes(cmax, b256::kClusterMax) : 0;
  return (int)((kClusterSmemBytes - lists) / (per_tile * (size_t)roles));
}

// Largest cluster (a power of two) the device takes for the cluster kernels: 16 where the opt-in
// for non-portable sizes is granted and such a cluster fits, else 8.  Asked once per device.
static int cluster_limit(int* out) {
  static std::mutex m;
  static int limit[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return ERSD_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(m);
  if (!limit[dev]) {
    constexpr int kKernels = 8;
    const void* kernels[kKernels] = {(const void*)b256::ersd_cluster_kernel<ERSD_BF16, 1>,
                                     (const void*)b256::ersd_cluster_kernel<ERSD_F32, 1>,
                                     (const void*)b256::ersd_cluster_kernel<ERSD_BF16, 2>,
                                     (const void*)b256::ersd_cluster_kernel<ERSD_F32, 2>,
                                     (const void*)b256::ersd_cluster_top_kernel<ERSD_BF16, 1>,
                                     (const void*)b256::ersd_cluster_top_kernel<ERSD_F32, 1>,
                                     (const void*)b256::ersd_cluster_top_kernel<ERSD_BF16, 2>,
                                     (const void*)b256::ersd_cluster_top_kernel<ERSD_F32, 2>};
    int lim = 16;
    for (int q = 0; q < kKernels; ++q) {
      e = cudaFuncSetAttribute(kernels[q], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kClusterSmemBytes);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    for (int q = 0; q < kKernels && lim == 16; ++q) {
      e = cudaFuncSetAttribute(kernels[q], cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      int n = 0;
      if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(16, 1, 1);
        cfg.blockDim = dim3(b256::kThreads, 1, 1);
        cfg.dynamicSmemBytes = kClusterSmemBytes;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = 16;
        at.val.clusterDim.y = 1;
        at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        e = cudaOccupancyMaxActiveClusters(&n, kernels[q], &cfg);
      }
      if (e != cudaSuccess || n < 1) lim = 8;
    }
    (void)cudaGetLastError();  // a refused opt-in only means clusters of eight
    limit[dev] = lim;
  }
  *out = limit[dev];
  return ERSD_OK;
}

// Whether a call can take a cluster kernel at all; cmax: most arrivals any of its races wants.
static bool cluster_applies(const Params& p, int dt, int cmax) {
  // (eight blocks, the portable cluster size, must be able to stage the rows of a position)
  const bool top = cmax > 1;
  const int roles = (p.mode == kVerify && p.draft) ? 2 : 1;
  const int64_t ntiles = ((int64_t)p.V + b256::kTile - 1) / b256::kTile;
  if (top && cmax > b256::kTopMaxC) return false;
  if (ntiles > 8 * (int64_t)cluster_max_tiles(dt, roles, cmax)) return false;
  if (top) {
    if (p.given_tok || p.chain_outputs || p.extra) return false;
  } else if (p.mode == kVerify && p.rows > 32) {
    return false;
  }
  return p.aligned_t && (roles == 1 || p.aligned_d) && p.rows <= 65535 && p.B <= 65535;
}

// Blocks per cluster.  Few positions: the smallest power of two that leaves a block about
// kClusterGroups tiles (shortest path through one position).  Once such clusters would make more
// than two blocks per SM: blocks of about twice as many tiles (measured at V = 128256: clusters
// of 8 beat clusters of 16 from about 20 positions on, clusters of 4 never beat clusters of 8).
static int cluster_size(const ersd_opts& o, const Params& p, int dt, int cmax, int* out) {
  int lim = 8;
  const int ls = cluster_limit(&lim);
  if (ls != ERSD_OK) return ls;
  const int ntiles = (p.V + b256::kTile - 1) / b256::kTile;
  const int roles = (p.mode == kVerify && p.draft) ? 2 : 1;
  const int max_tiles = cluster_max_tiles(dt, roles, cmax);
  if (o.split_v) {  // the caller's choice: a power of two that the device takes and whose blocks can stage their share
    const int CL = (int)o.split_v;
    if (CL > lim || (CL & (CL - 1)) != 0 || (ntiles + CL - 1) / CL > max_tiles) return ERSD_EUNSUPPORTED;
    *out = CL;
    return ERSD_OK;
  }
  int CL = 1;
  while (CL < lim && CL * b256::kClusterGroups < ntiles) CL *= 2;
  const int64_t units = (int64_t)p.B * p.rows;
  if (units * CL > 2 * sm_count() && CL > 1 && (CL / 2) * 2 * b256::kClusterGroups >= ntiles &&
      (ntiles + CL / 2 - 1) / (CL / 2) <= max_tiles)
    CL /= 2;
  *out = CL;
  return ERSD_OK;
}

// Whether a call that leaves the choice to the library takes the cluster kernel.
static bool cluster_by_default(const ersd_opts& o, const Params& p, int dt, int cmax) {
  if (o.kernel_path != 0 || o.split_v != 0 || o.block_threads != 0 || !cluster_applies(p, dt, cmax)) return false;
  int CL = 1;
  if (cluster_size(o, p, dt, cmax, &CL) != ERSD_OK) return false;
  const int64_t blocks = (int64_t)p.B * p.rows * CL;
  if (cmax > 1) return blocks <= kClusterAutoBlocksTop;
  if (p.mode == kVerify) {
    // counted in clusters of the size a lone position would get (16 blocks at V = 128256, 4 at
    // 32000), whatever size this call's clusters have: 44 and 176 positions at those two sizes
    const int ntiles = (p.V + b256::kTile - 1) / b256::kTile;
    int full = 1;
    while (full < b256::kClusterMax && full * b256::kClusterGroups < ntiles) full *= 2;
    return (int64_t)p.B * p.rows * full <= kClusterAutoBlocksVerify;
  }
  return blocks <= kClusterAutoBlocksSample;
}

template <int DT>
static int launch_cluster_dt(const ersd_opts& o, const Params& p_in, const TreeDesc& tree, int cmax, cudaStream_t st) {
  Params p = p_in;
  p.top_cmax = cmax;
  int roles = (p.mode == kVerify && p.draft) ? 2 : 1;
  int CL = 1;
  const int ls = cluster_size(o, p, DT, cmax, &CL);
  if (ls != ERSD_OK) return ls;
  const int ntiles = (p.V + b256::kTile - 1) / b256::kTile;
  // Trees of few positions: a cluster per ROW (a node's draft row and its target row side by side
  // in two clusters, each drawing the position's race variables) while all clusters are resident
  // at once; the longest chain of work in the call, the root's, is then half as long.
  int jobs = p.rows;
  if (cmax > 1 && roles == 2) {
    int with_children = 0;
    for (int n = 0; n < p.rows; ++n) with_children += tree.nchild[n] > 0 ? 1 : 0;
    const int64_t rows_in_all = (int64_t)p.B * (p.rows + with_children);
    bool split = rows_in_all * CL <= kClusterSplitBlocks;
    if (!split && !o.split_v && CL >= 2 && rows_in_all * (CL / 2) <= kClusterSplitBlocks &&
        (ntiles + CL / 2 - 1) / (CL / 2) <= cluster_max_tiles(DT, 1, cmax)) {
      CL /= 2;  // (a row to a cluster of half as many blocks)
      split = true;
    }
    if (split) {
      p.top_split = 1 + with_children;
      jobs = p.rows + with_children;
      roles = 1;
    }
  }
  const int G = (ntiles + CL - 1) / CL;  // tiles per block; they fit, see cluster_applies
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)CL, (unsigned)jobs, (unsigned)p.B);
  cfg.blockDim = dim3(b256::kThreads, 1, 1);
  cfg.dynamicSmemBytes = b256::cluster_role_bytes<DT>(G) * (size_t)roles + (cmax > 1 ? b256::top_list_bytes(cmax, CL) : 0);
  cfg.stream = st;
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeClusterDimension;
  at.val.clusterDim.x = (unsigned)CL;
  at.val.clusterDim.y = 1;
  at.val.clusterDim.z = 1;
  cfg.attrs = &at;
  cfg.numAttrs = 1;
  snprintf(g_last_launch, sizeof g_last_launch, "%s<%s, %d row(s) per cluster>: %d clusters of %d x %d threads, %d positions",
           cmax > 1 ? "ersd_cluster_top_kernel" : "ersd_cluster_kernel", DT == ERSD_BF16 ? "bf16" : "f32", roles,
           p.B * jobs, CL, b256::kThreads, p.B * p.rows);
  cudaError_t e;
  if (cmax > 1) {
    auto kernel = roles == 2 ? b256::ersd_cluster_top_kernel<DT, 2> : b256::ersd_cluster_top_kernel<DT, 1>;
    e = cudaLaunchKernelEx(&cfg, kernel, p, tree);
  } else {
    auto kernel = roles == 2 ? b256::ersd_cluster_kernel<DT, 2> : b256::ersd_cluster_kernel<DT, 1>;
    e = cudaLaunchKernelEx(&cfg, kernel, p);
  }
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

static int launch_cluster(const ersd_opts& o, const Params& p, const TreeDesc& tree, int dt, int cmax, cudaStream_t st) {
  return dt == ERSD_BF16 ? launch_cluster_dt<ERSD_BF16>(o, p, tree, cmax, st)
                         : launch_cluster_dt<ERSD_F32>(o, p, tree, cmax, st);
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
                       const ersd_opts* opts, void* stream, const int32_t* given_tok = nullptr,
                       bool check_only = false) {
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
  p.near_tie = o.near_tie_count;
  p.extra = o.near_tie_count ? 1 : 0;
  if (((uintptr_t)o.near_tie_count & 3) != 0) return ERSD_EALIGN;
  if (cmax + p.extra > ERSD_MAX_TOP_C) return ERSD_EUNSUPPORTED;
  cmax += p.extra;
  // sequences of few rows: one cluster per position (near-ties are counted by the streaming
  // kernel only: the cluster kernels keep no arrival beyond those asked for)
  if (o.kernel_path > 2) return ERSD_EINVAL;
  const bool cluster_ok = !p.extra && cluster_applies(p, dt, cmax);  // (a tree without branching is the chain 0 -> 1 -> ...)
  if (o.kernel_path == 2 && !cluster_ok) return ERSD_EUNSUPPORTED;
  if (o.block_threads != 0 && o.block_threads != 128 && o.block_threads != 256) return ERSD_EINVAL;
  if (o.workspace) {
    if (o.workspace_bytes < workspace_bytes(B, rows)) return ERSD_EWORKSPACE;
    if (((uintptr_t)o.workspace & 15) != 0) return ERSD_EALIGN;
  }
  if (check_only) return ERSD_OK;  // every host-side check has passed; nothing was enqueued
  void* ws = nullptr;
  const int st = get_workspace(o, workspace_bytes(B, rows), &ws, (cudaStream_t)stream);
  if (st != ERSD_OK) return st;
  p.slots = (Slot*)ws;
  if (cluster_ok && (o.kernel_path == 2 || cluster_by_default(o, p, dt, cmax)))
    return launch_cluster(o, p, tree, dt, cmax, (cudaStream_t)stream);
  int st0 = choose_threads(o, (int64_t)B * rows, &p.threads);
  if (st0 != ERSD_OK) return st0;
  set_chunks(p, choose_split(o, (int64_t)B * rows, V, cmax, p.threads));
  return launch(p, tree, dt, cmax, (cudaStream_t)stream);
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


// ---------------------------------------------------------------------------------------------
// Greedy speculative decoding (the paper's comparison verifier): kernels and launch logic.
// ---------------------------------------------------------------------------------------------
#include "ersd_gsd.inc"

// Scratch of a sequence-GSD call, carved from the front of the workspace: softmax statistics
// [B, 2k+1, 2] doubles, partial winners [B, S] (double, int), first rejections [B].
static size_t gsd_scratch_bytes(int64_t B, int64_t k, int64_t S) {
  return (size_t)(B * ((2 * k + 1) * 16 + S * 16 + 8));
}

static int gsd_check(const void* target, const void* draft, const int32_t* draft_tok, int dt,
                     const uint64_t* seeds, int B, int rows, int V, float T, const void* out_tokens,
                     const void* out_accept_len, bool need_draft) {
  int st = check_common(target, dt, seeds, B, rows, V, T);
  if (st != ERSD_OK) return st;
  if (!(T > 0.0f)) return ERSD_EINVAL;  // the ratio test needs softmax(z / T)
  if (!out_tokens || !out_accept_len) return ERSD_EINVAL;
  if (need_draft) {
    if (!draft || !draft_tok) return ERSD_EINVAL;
    if (((uintptr_t)draft & (elem_size(dt) - 1)) != 0 || ((uintptr_t)draft_tok & 3) != 0) return ERSD_EALIGN;
  }
  return ERSD_OK;
}

static void gsd_fill(GsdParams& g, const ersd_opts& o, const void* target, const void* draft,
                     const int32_t* draft_tok, const uint64_t* seeds, int B, int k, int V, float T,
                     int rows_t, int rows_d, int32_t* out_tokens, int32_t* out_accept_len) {
  memset(&g, 0, sizeof g);
  g.target = target;
  g.draft = draft;
  g.draft_tok = draft_tok;
  g.seeds = seeds;
  g.seq_ids = o.seq_ids;
  g.pos_offsets = o.pos_offsets;
  g.temps = o.temps;
  g.ts_b = o.temp_stride_b;
  g.ts_r = o.temp_stride_r;
  g.ld_t = o.ld_target ? o.ld_target : V;
  g.ld_d = o.ld_draft ? o.ld_draft : V;
  g.T = T;
  g.B = B;
  g.k = k;
  g.V = V;
  g.rows_t = rows_t;
  g.rows_d = rows_d;
  g.out_tokens = out_tokens;
  g.out_accept_len = out_accept_len;
  g.out_path = o.out_path;
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
  const int extra = o.near_tie_count ? 1 : 0;
  if (c + extra > ERSD_MAX_TOP_C) return ERSD_EUNSUPPORTED;
  if (((uintptr_t)o.near_tie_count & 3) != 0) return ERSD_EALIGN;
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
  p.near_tie = o.near_tie_count;
  p.extra = extra;
  if (o.kernel_path > 2) return ERSD_EINVAL;
  // (near-ties are counted by the streaming kernel only: the cluster kernels keep no arrival beyond those asked for)
  const bool cluster_ok = !extra && cluster_applies(p, dt, c);
  if (o.kernel_path == 2 && !cluster_ok) return ERSD_EUNSUPPORTED;
  TreeDesc tree;
  memset(&tree, 0, sizeof tree);
  if (cluster_ok && (o.kernel_path == 2 || cluster_by_default(o, p, dt, c)))
    return launch_cluster(o, p, tree, dt, c, (cudaStream_t)cuda_stream);
  st = choose_threads(o, (int64_t)B * R, &p.threads);
  if (st != ERSD_OK) return st;
  set_chunks(p, choose_split(o, (int64_t)B * R, V, c + extra, p.threads));
  if (p.S > 1) {
    void* ws = nullptr;
    st = get_workspace(o, workspace_bytes(B, R), &ws, (cudaStream_t)cuda_stream);
    if (st != ERSD_OK) return st;
    p.slots = (Slot*)ws;
  }
  return launch(p, tree, dt, c + extra, (cudaStream_t)cuda_stream);
}

static int verify_sequence(const void* target_logits, const void* draft_logits, int dt,
                           const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                           int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream,
                           bool check_only) {
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
                     out_tokens, out_accept_len, opts, cuda_stream, nullptr, check_only);
}

int ersd_verify(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream) {
  return verify_sequence(target_logits, draft_logits, dt, seeds, B, k, V, T, out_tokens, out_accept_len,
                         opts, cuda_stream, false);
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
  int st = noalloc_scratch(&scratch);
  if (st != ERSD_OK) return st;
  o.struct_size = sizeof o;
  o.workspace = scratch;
  o.workspace_bytes = kNoallocBytes;
  // every host-side argument check of ersd_verify first: a refused call puts nothing on the stream
  st = verify_sequence(target_logits, draft_logits, dt, seeds, B, k, V, T, out_tokens, out_accept_len, &o,
                       cuda_stream, true);
  if (st != ERSD_OK) return st;
  // The array keeps whatever the previous call left; the arrival counters (the first 16 bytes
  // of every slot this call uses) must start at zero.
  const cudaError_t e = cudaMemset2DAsync(scratch, sizeof(Slot), 0, 16, (size_t)B * ((size_t)k + 1),
                                          (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return verify_sequence(target_logits, draft_logits, dt, seeds, B, k, V, T, out_tokens, out_accept_len, &o,
                         cuda_stream, false);
}


int ersd_gsd_verify(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                    ersd_dtype dt, const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                    int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream) {
  if (k < 0) return ERSD_EINVAL;
  if (k + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  int st = gsd_check(target_logits, draft_logits, draft_tokens, dt, seeds, B, k + 1, V, T, out_tokens,
                     out_accept_len, k > 0);
  if (st != ERSD_OK) return st;
  const ersd_opts o = read_opts(opts);
  GsdParams g;
  gsd_fill(g, o, target_logits, draft_logits, draft_tokens, seeds, B, k, V, T, k + 1, k, out_tokens,
           out_accept_len);
  if (g.ld_t < V || g.ld_d < V) return ERSD_EINVAL;
  // slices of the final race: about two blocks per multiprocessor in all, at least 4096 tokens each
  int S = (2 * sm_count() + B - 1) / B;
  if (S > (V + 4095) / 4096) S = (V + 4095) / 4096;
  if (S > 64) S = 64;
  if (S < 1) S = 1;
  g.S = S;
  const size_t need = gsd_scratch_bytes(B, k, S);  // (never more than ersd_workspace_bytes(B, k + 1))
  void* ws = nullptr;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  st = get_workspace(o, workspace_bytes(B, k + 1), &ws, stream);
  if (st != ERSD_OK) return st;
  char* w = (char*)ws;
  g.stats = (double*)w;
  w += (size_t)B * (2 * k + 1) * 16;
  g.part_t = (double*)w;
  w += (size_t)B * S * 8;
  g.part_i = (int*)w;
  w += (size_t)B * S * 4;
  g.jstar = (int*)w;
  const dim3 rows_grid((unsigned)(2 * k + 1), (unsigned)B), race_grid((unsigned)S, (unsigned)B);
  const unsigned seq_blocks = (unsigned)((B + 127) / 128);
  if (dt == ERSD_BF16) {
    gsd_stats_kernel<ERSD_BF16><<<rows_grid, kGsdThreads, 0, stream>>>(g);
    gsd_scan_kernel<ERSD_BF16><<<seq_blocks, 128, 0, stream>>>(g);
    gsd_race_kernel<ERSD_BF16><<<race_grid, kGsdThreads, 0, stream>>>(g);
  } else {
    gsd_stats_kernel<ERSD_F32><<<rows_grid, kGsdThreads, 0, stream>>>(g);
    gsd_scan_kernel<ERSD_F32><<<seq_blocks, 128, 0, stream>>>(g);
    gsd_race_kernel<ERSD_F32><<<race_grid, kGsdThreads, 0, stream>>>(g);
  }
  gsd_finish_kernel<<<seq_blocks, 128, 0, stream>>>(g);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  // the workspace's resting state is all zero (the race kernels' arrival counters count on it)
  e = cudaMemsetAsync(ws, 0, need, stream);
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
}

int ersd_gsd_verify_tree(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                         ersd_dtype dt, const int32_t* parent, const uint64_t* seeds, int B, int N, int V,
                         float T, int32_t* out_tokens, int32_t* out_accept_len, const ersd_opts* opts,
                         void* cuda_stream) {
  if (N < 0 || !parent) return ERSD_EINVAL;
  if (N + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  int st = gsd_check(target_logits, draft_logits, draft_tokens, dt, seeds, B, N + 1, V, T, out_tokens,
                     out_accept_len, N > 0);
  if (st != ERSD_OK) return st;
  TreeDesc tree;
  int D = 0, cmax = 1;
  st = build_tree(parent, N, &tree, &D, &cmax);
  if (st != ERSD_OK) return st;
  const ersd_opts o = read_opts(opts);
  GsdParams g;
  gsd_fill(g, o, target_logits, draft_logits, draft_tokens, seeds, B, N, V, T, N + 1, N + 1, out_tokens,
           out_accept_len);
  if (g.ld_t < V || g.ld_d < V) return ERSD_EINVAL;
  g.depth = D;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (dt == ERSD_BF16) gsd_tree_kernel<ERSD_BF16><<<(unsigned)B, kGsdTreeThreads, 0, stream>>>(g, tree);
  else gsd_tree_kernel<ERSD_F32><<<(unsigned)B, kGsdTreeThreads, 0, stream>>>(g, tree);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? ERSD_OK : cuda_fail(e);
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

const char* ersd_last_launch(void) { return g_last_launch; }

int ersd_version(void) { return 111; }

}  // extern "C"
