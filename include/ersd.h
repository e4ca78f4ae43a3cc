/*
 * libersd -- exponential-race speculative decoding (ERSD) on one B200 (sm_100a).
 *
 * The library computes the data-parallel step of ERSD: for every draft and
 * target logit row, the winner (or the first c arrivals) of an exponential
 * race over the vocabulary, with the draft row and the target row of the same
 * position sharing one realisation of the race variables, and from those
 * winners the accepted prefix and the extra token.
 *
 * The race (Section 3 of the paper, "Exponential Races"): every token i gets
 * e_i ~ Exp(1); the winner under a law p is argmin_i e_i / p_i and is
 * distributed as p.  With p = softmax(logit / T) the library evaluates the
 * equivalent log form
 *
 *     key_i = ln e_i - logit_i / T,        winner = argmin_i key_i,
 *
 * which needs no softmax (ln(e_i/p_i) = key_i + ln Z, Z free of i).  The paper
 * names no random generator; here e_i = -log1p(-w_i), w_i = (x_i + 1/2) 2^-32,
 * with x_i word (i & 3) of Philox4x32-10 (Salmon et al. 2011) under key
 * (low, high 32 bits of seeds[b]) and counter (i >> 2, position, sequence id,
 * 0).  position = pos_offsets[b] + r (r = row index, or node id in a tree);
 * sequence id = b unless opts->seq_ids is given.  Exact key ties go to the
 * lowest token id.  A NaN logit counts as -inf; -inf never wins; a row in
 * which no token has positive probability yields token -1.
 *
 * Conventions for every call
 *   - Unless stated otherwise every data pointer is a DEVICE pointer to memory
 *     owned by the caller; the library never frees or keeps caller memory.
 *   - Logit tensors are row-major with the vocabulary contiguous.  Rows are
 *     `ld` elements apart (opts->ld_*; 0 means V) and row (b, r) starts at
 *     element (b * rows_per_sequence + r) * ld.  16-byte aligned rows take
 *     the vectorised path; other alignments are accepted and take a slower
 *     scalar path.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t, NULL = default
 *     stream) and never synchronise.  The return value is a host-side status:
 *     argument errors are found before anything is launched, launch errors
 *     are reported as ERSD_ECUDA (see ersd_last_cuda_error).
 *   - T is the temperature of every row unless opts->temps is given.  It must
 *     be finite and >= 0; T == 0 selects greedy decoding (key_i = -logit_i,
 *     no randomness).  A per-row temperature that is negative or not finite
 *     makes that row yield token -1.
 *   - Scratch memory: calls that split rows over several thread blocks, and
 *     every verify call, exchange partial results through a workspace.  Give
 *     one in opts->workspace (size from ersd_workspace_bytes, zeroed once
 *     with ersd_workspace_init; every call leaves it ready for the next
 *     call, of any size that fits): then the call allocates nothing and only
 *     enqueues work on `cuda_stream`.  Or pass none and the library keeps ONE
 *     private workspace per device.  Two things follow from that.  (1) A call
 *     that needs more than the private workspace holds makes it grow with
 *     cudaFree and cudaMalloc, which synchronise the whole device, and zeroes
 *     it on `cuda_stream`; such a call is not asynchronous and cannot be part
 *     of a stream capture.  (2) Every call on the device that passes no
 *     workspace uses that same memory, whatever its stream: such calls must
 *     not overlap on the GPU.  Calls that may overlap (different streams,
 *     host threads without ordering between them) each need a workspace of
 *     their own in opts->workspace; sharing one gives wrong results.
 *   - Randomness contract: a (seed, sequence id, position) triple must not be
 *     reused for two EMITTED tokens.  Reusing the positions of a rejected
 *     speculation in the next round is fine: what is emitted depends only on
 *     races at positions up to the first disagreement.
 */
#ifndef ERSD_H_
#define ERSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { ERSD_F32 = 0, ERSD_BF16 = 1 } ersd_dtype;

typedef enum {
  ERSD_OK = 0,
  ERSD_EINVAL = -1,       /* bad argument (null pointer, size out of range, bad T, bad tree) */
  ERSD_EALIGN = -2,       /* pointer not aligned to its element size */
  ERSD_EUNSUPPORTED = -3, /* size beyond a compiled limit (see ERSD_MAX_*) */
  ERSD_ECUDA = -4,        /* a CUDA runtime call failed; see ersd_last_cuda_error() */
  ERSD_EWORKSPACE = -5,   /* opts->workspace given but too small */
  ERSD_ENOALLOC_LIMIT = -6 /* ersd_verify_noalloc: B * (k + 1) > ERSD_NOALLOC_MAX_ROWS */
} ersd_status;

#define ERSD_MAX_TOP_C 64   /* arrivals per race (children per tree node, opts->top_c) */
#define ERSD_MAX_ROWS 256   /* rows per sequence: k + 1, N + 1 */
#define ERSD_MAX_SPLIT 32   /* thread blocks sharing one row */
#define ERSD_NOALLOC_MAX_ROWS 1024 /* ersd_verify_noalloc: largest B * (k + 1) */

/* Optional arguments.  Pass NULL for defaults.  Set struct_size = sizeof(ersd_opts). */
typedef struct ersd_opts {
  uint32_t struct_size;
  uint32_t top_c;          /* ersd_race_sample: arrivals per row, 0 or 1 = winner only */
  uint32_t split_v;        /* thread blocks per row (cluster kernel: per cluster, a power of two up to 16);
                              0 = chosen by the library */
  uint32_t block_threads;  /* threads per block of the race kernel: 128, 256, or 0 = chosen by the library */
  int64_t ld_target;       /* row stride in elements of target_logits / logits; 0 = V */
  int64_t ld_draft;        /* row stride in elements of draft_logits; 0 = V */
  const float* temps;      /* device; temperature of row (b, r) = temps[b*temp_stride_b + r*temp_stride_r] */
  int64_t temp_stride_b;
  int64_t temp_stride_r;
  const uint32_t* seq_ids;     /* device [B]; NULL: sequence id = b */
  const uint32_t* pos_offsets; /* device [B]; NULL: 0 */
  int32_t* out_draft_tok;  /* device, nullable.  verify: [B, k], entry j = token drafted at position j.
                              verify_tree: [B, N+1], entry n = token drafted at node n (entry 0 = -1). */
  float* out_draft_key;    /* device, nullable, same shape: race key of that drafted token */
  int32_t* out_target_tok; /* device, nullable, [B, k+1] / [B, N+1]: target winner of every row */
  float* out_target_key;   /* device, nullable, same shape: its race key */
  int32_t* out_path;       /* device, nullable, verify_tree: [B, D+1] accepted node ids, -1 padded */
  float* out_key;          /* device, nullable, ersd_race_sample: [B, R, c] keys of the arrivals */
  void* workspace;         /* device scratch or NULL (library-owned) */
  size_t workspace_bytes;
  uint32_t kernel_path;    /* ersd_race_sample, ersd_verify, ersd_verify_tokens, ersd_verify_noalloc,
                              ersd_verify_tree:
                              0 = chosen by the library, 1 = the streaming kernel, 2 = a cluster kernel
                              (one thread-block cluster per position, for calls of few rows; one kernel for
                              races of one arrival, one for races of up to 32: top_c > 1, trees with
                              branching;
                              ERSD_EUNSUPPORTED where neither applies: a race of more than 32 arrivals,
                              rows not 16-byte aligned, B or R > 65535, more than 32 rows per sequence
                              in ersd_verify and its variants, near_tie_count given, or a vocabulary too
                              long for eight blocks to stage in shared memory: beyond about 320 k entries
                              in bf16, 160 k in fp32, halved when draft rows are raced along, less the
                              room the lists of a race of several arrivals take) */
  uint32_t reserved1;
  uint32_t* near_tie_count; /* device, nullable: a counter the call ADDS to (the caller zeroes it): the number
                              of races in which two consecutive arrivals among the first c + 1 (c = arrivals
                              wanted: 1 for a winner, a node's child count for its draft row, top_c) have race
                              keys closer than 1e-5 -- the window inside which a reference in other arithmetic
                              may order the two the other way.  To see the runner-up every
                              race is run for one more arrival (c + 1 <= ERSD_MAX_TOP_C, else
                              ERSD_EUNSUPPORTED), which costs time, and the call takes the streaming kernel
                              (kernel_path 2 is refused).  Leave NULL in production. */
} ersd_opts;

/*
 * Race sampling (Section 3; the drafting lines of Algorithms 2 and 5).
 * For every sequence b < B and row r < R: out_tok[b, r, 0..c) = the first c
 * arrivals (c = max(1, opts->top_c), ascending key; -1 where fewer than c
 * tokens have positive probability) of the race of position
 * pos_offsets[b] + r under softmax(logits[b, r, :] / T).  The ordered
 * arrivals are a sample without replacement, which is how batch and tree
 * drafting pick sibling tokens.
 *   logits  device [B, R, V] of dtype dt       seeds   device [B] uint64
 *   out_tok device [B, R, c] int32
 * Errors: ERSD_EINVAL for null pointers, B, R, V < 1 or B * R beyond 2^31 - 1,
 * T < 0 or not finite; ERSD_EUNSUPPORTED for c > ERSD_MAX_TOP_C,
 * V > 0x7FFF0000, or more than 65535 rows per sequence or thread blocks per
 * row (the launch grid is (B, rows, blocks per row); fold rows into B -- with
 * opts->seq_ids and opts->pos_offsets naming each row's race -- to sample more
 * rows of one sequence in a call); ERSD_EALIGN.
 */
int ersd_race_sample(const void* logits, ersd_dtype dt, const uint64_t* seeds, int B, int R, int V,
                     float T, int32_t* out_tok, const ersd_opts* opts, void* cuda_stream);

/*
 * Sequence ERSD verification (Algorithm 2, extended to k drafted positions as
 * Section 3 describes: one race per position, accept in order until the first
 * disagreement).  For every sequence b and position j:
 *   draft_tok[j]  = winner of race (b, j) under draft row j            (j < k)
 *   target_tok[j] = winner of the SAME race under target row j         (j <= k)
 *   L = first j < k with draft_tok[j] != target_tok[j] (or target_tok[j] = -1), else k
 *   out_tokens[b, 0..L] = target_tok[0..L], out_tokens[b, j > L] = -1,
 *   out_accept_len[b] = L   (L + 1 tokens are emitted, between 1 and k + 1).
 *   target_logits device [B, k+1, V]    draft_logits device [B, k, V] (may be NULL when k = 0)
 *   seeds device [B] uint64   out_tokens device [B, k+1] int32   out_accept_len device [B] int32
 * Everything runs in one kernel launch.  Errors as above; k + 1 > ERSD_MAX_ROWS
 * is ERSD_EUNSUPPORTED.
 */
int ersd_verify(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream);

/*
 * Tree ERSD verification (Algorithm 5; batch drafting is the depth-1 tree).
 * The draft tree has nodes 0..N, node 0 the root (the current context).
 * `parent` is a HOST array [N+1] with parent[0] = -1 and 0 <= parent[n] < n.
 * Siblings are ordered by node id; the sibling of rank r (0-based) is taken
 * to carry the (r+1)-th arrival of its parent's race under the parent's
 * draft row.  Node n's race is the race of position pos_offsets[b] + n.
 * Walk: cur = root; emit the winner of cur's race under target row cur; move
 * to the child that drafted this token; stop when there is none.
 *   target_logits device [B, N+1, V], row n = target law after the path to node n
 *   draft_logits  device [B, N+1, V], row n = draft law after that path; rows of
 *                 leaves are never read
 *   out_tokens device [B, D+1] int32 (-1 padded), D = ersd_tree_depth(parent, N)
 *   out_accept_len device [B] int32 = number of drafted tokens accepted
 * Errors as above; a malformed parent array is ERSD_EINVAL; N + 1 > ERSD_MAX_ROWS
 * or a node with more than ERSD_MAX_TOP_C children is ERSD_EUNSUPPORTED.
 */
int ersd_verify_tree(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                     const int32_t* parent, const uint64_t* seeds, int B, int N, int V, float T,
                     int32_t* out_tokens, int32_t* out_accept_len, const ersd_opts* opts,
                     void* cuda_stream);

/*
 * Verification of tokens drafted earlier (Algorithm 2's verification lines on a
 * drafted sequence, Section 3: accept in order until the first rejection).
 * In a decoding loop the draft tokens already exist when the target model has
 * run -- they were produced one position at a time with ersd_race_sample on
 * the draft model's rows -- so only the target rows need to be raced:
 * half the bytes of ersd_verify, same result as long as the tokens were
 * drafted with the same (seed, sequence id, position) races.
 *   target_logits device [B, k+1, V]      draft_tokens device [B, k] int32
 *   out_tokens    device [B, k+1] int32   out_accept_len device [B] int32
 * Position j < k is accepted iff its target winner equals draft_tokens[b, j];
 * outputs as for ersd_verify.  opts->out_target_tok / out_target_key are
 * filled if given; opts->out_draft_tok echoes draft_tokens, out_draft_key is
 * filled with +inf.
 * Errors as for ersd_verify (draft_tokens may be NULL only when k == 0).
 */
int ersd_verify_tokens(const void* target_logits, const int32_t* draft_tokens, ersd_dtype dt,
                       const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                       int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream);

/*
 * Greedy speculative decoding (GSD) on the same logits -- the verifier the paper
 * compares ERSD with (Algorithm 1, Section 2, applied position by position:
 * drafted tokens are verified in order until the first rejection).  For every
 * sequence b and position j < k, in order:
 *   x = draft_tokens[b, j], a sample of softmax(draft row j / T) made earlier
 *       (any sampler; ersd_race_sample on the draft rows is one);
 *   accept iff P_j(x) / Q_j(x) > u, with P_j, Q_j the softmax of target / draft
 *       row j and u ~ Uniform(0, 1);
 *   on the first rejection emit a sample of max(P_j - Q_j, 0) / sum and stop;
 *   after k acceptances emit a sample of softmax(target row k / T).
 * Randomness (the paper names none): u is word 0 of Philox4x32-10 under the
 * sequence's key with counter (0, position, sequence id, 1), u = (x + 1/2) 2^-32;
 * the token that ends the call is the winner of an exponential race over the
 * residual (or target) law, argmin_i e_i / w_i, with e_i from counter
 * (i >> 2, position, sequence id, 2) -- both independent of the drafting races
 * (last counter word 0), as Algorithm 1 requires.  All arithmetic is double
 * precision; the call is four small launches, not the single streaming launch
 * of ersd_verify.
 *   target_logits device [B, k+1, V]   draft_logits device [B, k, V]
 *   draft_tokens  device [B, k] int32  out_tokens device [B, k+1] int32 (-1 padded)
 *   out_accept_len device [B] int32
 * opts: ld_*, temps (every temperature must be > 0), seq_ids, pos_offsets,
 * workspace (ersd_workspace_bytes(B, k + 1) bytes, as for ersd_verify; left zeroed).
 * Errors as for ersd_verify; T <= 0 is ERSD_EINVAL (the test needs a softmax).
 */
int ersd_gsd_verify(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                    ersd_dtype dt, const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                    int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream);

/*
 * Tree GSD (Algorithm 4, Appendix A; the algorithm is printed with the tested
 * token's child index missing and an empty loop -- the reading taken is Section
 * 2's text: recursive batch selection).  Tree layout as for ersd_verify_tree
 * (`parent` a HOST array).  draft_tokens[b, n] is the token drafted at node n
 * (entry 0 unused); siblings must have been drafted WITHOUT replacement from
 * their parent's draft row (the first arrivals of ersd_race_sample with top_c
 * are).  Walk from the root: the current node's children are tried in order;
 * child of rank i is accepted iff P_t(x) / Q_d(x) > u(node, i), where every
 * rejection replaces P_t by max(P_t - Q_d, 0) / sum and removes the rejected
 * token from Q_d (renormalised); an accepted child becomes the current node with
 * its own rows; when no child is accepted, or at a leaf, a sample of the current
 * P_t is emitted and the call ends.  u(node, i): counter (i, node, sequence id, 1);
 * the final race: counter (token >> 2, node, sequence id, 2).
 *   target_logits, draft_logits device [B, N+1, V] (draft rows of leaves never read)
 *   draft_tokens device [B, N+1] int32   out_tokens device [B, D+1] int32 (-1 padded)
 *   out_accept_len device [B] int32      opts->out_path as for ersd_verify_tree
 * One thread block walks one sequence, in double precision: a comparison path,
 * not a throughput path.
 */
int ersd_gsd_verify_tree(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                         ersd_dtype dt, const int32_t* parent, const uint64_t* seeds, int B, int N, int V,
                         float T, int32_t* out_tokens, int32_t* out_accept_len, const ersd_opts* opts,
                         void* cuda_stream);

/*
 * ersd_verify for callers that must not allocate device memory.  (The paper has
 * no counterpart; this is a deployment variant of ersd_verify and computes
 * exactly the same outputs from the same arguments.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * serving loop whose memory is fully pre-planned by a pool allocator, in a
 * latency-critical section where the implicit device synchronisation of
 * cudaMalloc/cudaFree is unacceptable, or in a process whose device memory is
 * already handed out to the last byte.  ersd_verify either wants a workspace
 * from the caller or grows a private one with cudaMalloc; this entry point does
 * neither.  Its scratch is a fixed array of about 2.1 MB compiled into the
 * library image (every GPU that loads the library holds that much until the
 * process exits), sized for B * (k + 1) <= ERSD_NOALLOC_MAX_ROWS.  Larger calls
 * are refused with ERSD_ENOALLOC_LIMIT and nothing is launched.  The call makes
 * no cudaMalloc, cudaFree or other allocating call.
 *
 * Arguments, outputs and errors are those of ersd_verify, except that
 * opts->workspace must be NULL (ERSD_EINVAL otherwise).
 *
 * First call on a device: the library looks up the array's device address
 * (once per device, with the caller's current device) before it launches.
 * Make that first call outside any stream capture; a throw-away call at
 * start-up is enough.
 *
 * Sharing: every call on a device uses the same array, which still holds what
 * the previous call left there.  The library clears the part that must start
 * at zero on `cuda_stream` before each launch.  Two calls that can overlap on
 * the GPU (different streams, or different host threads without ordering
 * between them) race on the array and give wrong results; serialise them, or
 * use ersd_verify with one workspace per stream.
 */
int ersd_verify_noalloc(const void* target_logits, const void* draft_logits, ersd_dtype dt,
                        const uint64_t* seeds, int B, int k, int V, float T, int32_t* out_tokens,
                        int32_t* out_accept_len, const ersd_opts* opts, void* cuda_stream);

/*
 * Draft tree with the largest expected number of accepted tokens (Algorithm 3,
 * "Optimal tree construction", Section 4).  HOST function, no GPU work.
 * Acceptance probabilities follow the 0-th order model of the paper's
 * experiments: a vertex reached through child ranks (j_1, .., j_m) is accepted
 * with probability accept[j_1] * ... * accept[j_m], where accept[r] (HOST array
 * of max_children doubles in [0, 1], non-increasing in r) is the probability
 * that a verified node's child of rank r -- the (r+1)-th arrival of its race
 * under the draft row -- is accepted.  Vertices are added greedily by
 * probability from a priority queue; a chosen vertex offers its first child and
 * its next sibling (ties: shallower first, then lexicographic).
 *   parent_out  HOST [k + 1]: parent_out[0] = -1, vertices in lexicographic
 *               order, so parent_out[n] < n and siblings ascend by rank -- the
 *               form ersd_verify_tree takes.
 *   expected_tokens  HOST, nullable: sum of the k vertices' probabilities.
 * Errors: ERSD_EINVAL (null pointers, k < 0, max_children < 1, accept outside
 * [0, 1] or increasing); ERSD_EUNSUPPORTED for k + 1 > ERSD_MAX_ROWS.  Ranks
 * beyond ERSD_MAX_TOP_C are ignored.
 */
int ersd_optimal_tree(const double* accept, int max_children, int k, int32_t* parent_out,
                      double* expected_tokens);

/*
 * Empirical acceptance profile for ersd_optimal_tree (Section 5 of the paper: the
 * acceptance probability function R is estimated from observed acceptances and
 * treated as a 0-th order Markov source).  HOST function, no GPU work.
 *   paths   HOST [B, D+1]: accepted node ids per sequence, -1 padded -- what
 *           opts->out_path of ersd_verify_tree (or ersd_gsd_verify_tree) returns,
 *           copied to the host; D = ersd_tree_depth(parent, N)
 *   parent  HOST [N+1]: the draft tree those calls verified
 *   accept  HOST [max_children] out: accept[r] = (times a child of rank r was the
 *           accepted one) / (times a node with a child of rank r was verified);
 *           0 where never tried; capped so that it never rises with r, the form
 *           ersd_optimal_tree takes
 *   trials  HOST [max_children] out, nullable: the denominators
 * Errors: ERSD_EINVAL (null pointers, malformed parent array, a path that is not
 * a root path of the tree); ERSD_EUNSUPPORTED for N + 1 > ERSD_MAX_ROWS.
 */
int ersd_acceptance_profile(const int32_t* paths, const int32_t* parent, int B, int N, int max_children,
                            double* accept, int64_t* trials);

/* Depth (longest root-to-leaf edge count) of a HOST parent array, or -1 if it is malformed. */
int ersd_tree_depth(const int32_t* parent, int N);

/*
 * Race keys of one row, for diagnostics and tests (Section 3, key_i as above,
 * natural-log units): out_keys[i], i < V, device float32.
 *   mode 0: the double-precision evaluation the library uses to decide winners;
 *   mode 1: the single-precision screening value it uses to discard losers
 *           (within about 1e-3 of mode 0 for |key| up to a few hundred);
 *   mode 2: (mode-0 key minus the same key formed with the CUDA math library's
 *           log and log1p) * 1e12 -- checks the library's own straight-line
 *           double-precision logarithm on the device.
 */
int ersd_row_keys(const void* row_logits, ersd_dtype dt, int V, float T, uint64_t seed,
                  uint32_t seq_id, uint32_t position, int mode, float* out_keys, void* cuda_stream);

/* Bytes of scratch that any call with these sizes can need. */
size_t ersd_workspace_bytes(int B, int rows_per_seq);
/* Zero a caller-owned workspace (needed once, before its first use). */
int ersd_workspace_init(void* workspace, size_t bytes, void* cuda_stream);

const char* ersd_status_string(int status);
int ersd_last_cuda_error(void); /* cudaError_t of the last failing runtime call on this thread */
/* Which kernel this thread's last ersd_race_sample / ersd_verify* call launched and in what shape
   (a short text for logs and benchmarks; "" before the first launch).  Diagnostic only. */
const char* ersd_last_launch(void);
int ersd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ERSD_H_ */
