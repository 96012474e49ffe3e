/*
 * gto.h - C ABI of the B200 draft-tree pass of Group Tree Optimization (GTO).
 *
 * One training micro-batch holds B positions.  For every position there are G = 2
 * draft trees: t = 0 built from the current draft model's logits, t = 1 from the
 * frozen reference draft's.  Logit rows are inputs (one V-wide row per context):
 *
 *   draft  [G, B, D, k, V_draft]   row [t,b,0,0,:] is the root context; row [t,b,d,j,:]
 *                                  (1 <= d < D) is the context reached through frontier
 *                                  slot j of depth d; rows [t,b,0,1..k-1,:] are never read.
 *   target [G, B, R, V_target]     R = 1 + (D-1)*k; row 0 = root context, row
 *                                  1 + (d-1)*k + j = frontier slot j of depth d.
 *
 * Logits are bf16, fp16 (the paper trains under FP16 autocast, App. B) or fp32, row-major,
 * contiguous; V_draft and V_target must make a row a
 * multiple of 16 bytes.  All pointers in the structs below are DEVICE pointers owned by
 * the caller, 16-byte aligned, dense row-major with the shapes given.  The library
 * allocates memory only in gto_create (its device workspace and a page-locked host copy of
 * the row list for gto_tree_reward_host) and keeps no caller pointer
 * after a call returns.  Calls enqueue work on `stream` (a cudaStream_t passed as void*)
 * and return without synchronising; argument errors are returned at once and launch
 * nothing.  Data faults (a non-finite row sum, an index out of range in a caller's table) are recorded
 * in a device status word read by gto_device_status.  A context is not thread-safe;
 * use one per host thread and device.  No entry point writes to stdout or throws.
 */
#ifndef GTO_H_
#define GTO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gto_ctx gto_ctx; /* opaque; owns the workspace only */

typedef enum {
  GTO_OK = 0,
  GTO_ERR_INVALID_ARG = 1, /* null pointer, bad shape, misaligned pointer               */
  GTO_ERR_UNSUPPORTED = 2, /* shape outside the compiled limits (see gto_create)        */
  GTO_ERR_WORKSPACE = 3,   /* workspace allocation failed                                */
  GTO_ERR_CUDA = 4,        /* a CUDA runtime call failed                                 */
  GTO_ERR_NONFINITE = 5,   /* device status: a row's log-sum-exp was not finite          */
  /* 6 is not used: no kernel of the library waits on anything                            */
  GTO_ERR_TOO_LARGE = 7,   /* gto_build_tree_noalloc: batch exceeds the fixed scratch    */
  GTO_ERR_BAD_INDEX = 8    /* device status: an index in a caller's table (d2t, a tree's
                              rows, tokens or parents, a path's rows) was out of range; the
                              entry was skipped, results that depend on it are unspecified  */
} gto_status;

typedef enum { GTO_F32 = 0, GTO_BF16 = 1, GTO_F16 = 2 } gto_dtype;

/* Reward aggregation over the tree's sequences: Eq. 5 (log-sum-exp smooth max, the
 * default) or the two alternatives of the aggregation ablation in Sec. 4.2. */
typedef enum { GTO_AGG_LSE = 0, GTO_AGG_MAX = 1, GTO_AGG_MEAN = 2 } gto_agg;

enum {
  GTO_FLAG_STD_UNBIASED = 1u, /* Eq. 10 with the sample std (divide by m-1)             */
  GTO_FLAG_NO_DEBIAS = 2u,    /* Eq. 9 switched off: R_i = r(T_i) (debiasing ablation)  */
  GTO_FLAG_FORCE_ROW_SPLIT = 16u, /* always split a logit row over a thread-block cluster (the
                                  library does so by itself where it pays: few, long rows);
                                  for tests and tuning                                      */
  GTO_FLAG_SEQ_ALL_NODES = 8u, /* Eq. 5 over the root-to-node sequence of every selected node
                                  instead of the root-to-leaf sequences only                 */
  GTO_FLAG_PATH_MAX_EXPECTED = 32u, /* the "longest accepted sequence" of Sec. 3.2 read as the
                                  candidate sequence with the largest expected acceptance length
                                  L_i of Eq. 3 (lowest list position on ties), reported whole, root
                                  to its last node; default: the greedy-target verification walk */
  GTO_FLAG_GRAD_LIVE_ROWS = 4u /* gto_group_surrogate_grad writes only the rows that carry a
                                  gradient (j < path_len[b] and coeff[b] != 0) and leaves the
                                  rest of grad untouched, instead of filling it with zeros   */
};

typedef struct {
  int32_t B;        /* positions; a multiple of m                                       */
  int32_t G;        /* trees per position; must be 2                                    */
  int32_t D;        /* maximum tree depth d of Sec. 3.1                                 */
  int32_t k;        /* top-k per node expansion and per layer (App. B: 10)              */
  int32_t g;        /* nodes kept by the global prune, root excluded (App. B: 60)       */
  int32_t m;        /* group size of Eq. 6 (App. B: 8); groups are consecutive positions */
  int32_t V_draft;  /* draft vocabulary                                                  */
  int32_t V_target; /* target vocabulary                                                 */
  int32_t logit_dtype; /* gto_dtype of draft, target and grad                           */
  int32_t reward_agg;  /* gto_agg                                                       */
  float eta;        /* smooth-max temperature of Eq. 5 (App. B: 1)                      */
  float clip_eps;   /* epsilon of Eq. 12                                                */
  float std_delta;  /* delta of Eq. 10                                                  */
  float grad_scale; /* factor on the summed group losses (a trainer passes omega / K)   */
  uint32_t flags;
} gto_config;

/* The pruned draft trees (Sec. 3.1, tree policy G).  Node lists hold g nodes per tree in
 * ascending pool index (depth-major candidate number), so a parent precedes its children. */
typedef struct {
  int32_t* node_token;   /* [G,B,g] draft-vocabulary id                                  */
  int32_t* node_parent;  /* [G,B,g] list position of the parent, -1 = child of the root  */
  int32_t* node_depth;   /* [G,B,g] 1..D                                                 */
  int32_t* node_ctx_row; /* [G,B,g] context row (0..R-1) the token was proposed from     */
  int32_t* node_slot;    /* [G,B,g] frontier slot of the node at its depth, -1 = not expanded */
  int32_t* node_pool;    /* [G,B,g] pool index: c at depth 1, k + (d-2)k^2 + j*k + c later */
  float* node_logp;      /* [G,B,g] draft log-probability of the edge into the node      */
  double* node_score;    /* [G,B,g] global acceptance score: sum of node_logp on the path */
  uint64_t* node_mask;   /* [G,B,g,W] W = ceil(g/64): bit a of row n = a is n or an ancestor */
  double* row_lse;       /* [G,B,R] log-sum-exp of every draft context row               */
} gto_tree;

/* Draft Tree Reward (Eq. 3-5) and the longest accepted sequence (Sec. 3.2) of tree 0. */
typedef struct {
  double* reward;        /* [G,B] r = R(T; eta)                                          */
  double* etree;         /* [G,B] sum over nodes of the path product (exact expected
                                  accepted tokens under target sampling; auxiliary)      */
  int32_t* n_leaves;     /* [G,B] number N of sequences (leaves) in Eq. 5                */
  float* node_ptarget;   /* [G,B,g] target probability of the node's token in its context */
  float* node_pathprod;  /* [G,B,g] Eq. 4: product of node_ptarget from the root         */
  float* node_L;         /* [G,B,g] Eq. 3 for the sequence ending at the node            */
  double* row_lse_t;     /* [G,B,R] target log-sum-exp; NaN for rows no node uses        */
  int32_t* row_argmax_t; /* [G,B,R] greedy target token (lowest id on ties); -1 likewise */
  int32_t* path_len;     /* [B] l_i: accepted draft tokens of tree 0 under the greedy target */
  int32_t* path_node;    /* [B,D] list positions of the accepted nodes; -1 beyond l_i    */
  int32_t* path_row;     /* [B,D] context row of each step (the draft row that produced it) */
  int32_t* path_token;   /* [B,D] draft token ids                                        */
  float* path_logp;      /* [B,D] draft log-probability of each step; 0 beyond l_i       */
} gto_reward;

/* Group statistics and surrogate of Eq. 9-12. */
typedef struct {
  double* R;        /* [B] debiased reward, Eq. 9                                        */
  double* adv;      /* [B] standardised advantage, Eq. 10                                */
  double* ratio;    /* [B] s_i of Eq. 11                                                 */
  double* coeff;    /* [B] factor on (onehot - softmax) for every step of position i     */
  int32_t* active;  /* [B] 1 if the unclipped branch of Eq. 12 is the minimum            */
  double* loss;     /* [B/m] group losses of Eq. 12                                      */
} gto_grad_stats;

/* Validates the configuration and allocates the workspace on `device`.
 * Limits: G == 2; 1 <= k and k*k <= 128; 1 <= g <= min(128, k + (D-1)k^2); 1 <= D <= 16;
 * B % m == 0; G*B <= 65535; k <= V_draft; V * sizeof(logit) a multiple of 16 for both vocabularies.
 * Returns GTO_ERR_UNSUPPORTED outside them. */
gto_status gto_create(gto_ctx** ctx, const gto_config* cfg, int device);
gto_status gto_destroy(gto_ctx* ctx);

/* Tree policy G of Sec. 3.1 for all G*B trees: per context row the draft log-softmax and
 * its k best tokens (value descending, id ascending); layer-wise expansion keeping the k
 * best of the k*k candidates of each layer by cumulative log-probability (Fig. 1 caption:
 * path confidence is the product of edge probabilities); global top-g over all
 * k + (D-1)k^2 candidates.  Every tie goes to the lower index.  Writes every array of *out. */
gto_status gto_build_tree(gto_ctx* ctx, const void* draft_logits, const gto_tree* out,
                          void* stream);

/* Largest G*B*R*k (draft context rows times top-k) gto_build_tree_noalloc accepts: its
 * scratch is a fixed array of 8 bytes per entry (8 MiB) inside the library image. */
#define GTO_NOALLOC_MAX_ENTRIES (1 << 20)

/* gto_build_tree for callers that must not allocate device memory (no counterpart in the
 * paper: it is an integration aid).  A trainer that routes every device byte through its own
 * allocator, a process living inside a fixed memory budget, or a thread that cannot afford
 * the device-wide stall an allocation may cause, cannot create a gto_ctx, because gto_create
 * calls cudaMalloc.  This call needs no context: it takes the configuration directly and
 * keeps the per-row top-k tables in a fixed device array that ships with the library (every
 * GPU that loads the library holds those 8 MiB until the process ends).  It never calls
 * cudaMalloc, cudaFree or any allocating routine.
 *   - Computes exactly what gto_build_tree computes and writes every array of *out; only
 *     B, G, D, k, g, V_draft and logit_dtype of *cfg are used.
 *   - Returns GTO_ERR_TOO_LARGE when G*B*R*k > GTO_NOALLOC_MAX_ENTRIES: split the batch.
 *   - The first call on a device looks up the array's device address (one
 *     cudaGetSymbolAddress, cached per device); make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array and it keeps the last call's contents; the
 *     call clears what it needs cleared.  Two calls whose kernels can overlap on the GPU
 *     (different streams, no dependency between them) race on it: order them.
 *   - There is no status word to read back: a row with non-finite logits shows as a
 *     non-finite entry of out->row_lse. */
gto_status gto_build_tree_noalloc(const gto_config* cfg, int device, const void* draft_logits,
                                  const gto_tree* out, void* stream);

/* Draft Tree Reward, Eq. 3-5, and the longest accepted sequence of Sec. 3.2.  Reads only
 * the target rows that are the context of a selected node.  d2t maps draft ids to target
 * ids ([V_draft] int32, device, injective); NULL means identity and needs
 * V_draft == V_target.  Writes every array of *out. */
gto_status gto_tree_reward(gto_ctx* ctx, const gto_tree* tree, const void* target_logits,
                           const int32_t* d2t, const gto_reward* out, void* stream);

/* gto_tree_reward for target logits that live in HOST memory (Eq. 3-5 and Sec. 3.2 as
 * above).  Only the target rows that are the context of a selected node are needed
 * (about a fifth of them at the paper's tree shape), so only those cross the bus: the call
 * builds the row list on the device, reads it back (it SYNCHRONISES `stream` once), copies
 * each run of adjacent needed rows from target_host to the same offset of target_dev, and
 * then proceeds as gto_tree_reward on target_dev.  target_host: HOST [G,B,R,V_target],
 * should be page-locked for the copies to be asynchronous; target_dev: DEVICE scratch of the
 * same shape owned by the caller, rows that are not needed are left untouched.
 * *rows_copied (optional, host) receives the number of rows copied. */
gto_status gto_tree_reward_host(gto_ctx* ctx, const gto_tree* tree, const void* target_host,
                                void* target_dev, const int32_t* d2t, const gto_reward* out,
                                void* stream, int64_t* rows_copied);

/* Eq. 9-12 and the derivative of the summed group losses with respect to the draft logits:
 * grad[b,j,:] = coeff_b * (onehot(path_token[b,j]) - softmax(draft row path_row[b,j] of
 * tree 0)) for j < path_len[b], zero otherwise (also when the ratio is clipped).  With
 * GTO_FLAG_GRAD_LIVE_ROWS the zero rows are not written (a trainer that scatters the rows
 * into its logit gradient by path_row reads only the live ones).
 * old_logp [B,D] fp32: log-probabilities of the accepted tokens under the old / reference
 * draft (entries beyond path_len ignored).  grad [B,D,V_draft] in the logit dtype. */
gto_status gto_group_surrogate_grad(gto_ctx* ctx, const void* draft_logits,
                                    const gto_tree* tree, const gto_reward* reward,
                                    const float* old_logp, void* grad,
                                    const gto_grad_stats* out, void* stream);

/* Token-level loss of Eq. 13 / App. B. */
typedef struct {
  double* loss;   /* [B] H(p_T, p_M) of the position's prefix                              */
  double* lse_t;  /* [B] log-sum-exp of the target logits over the (mapped) draft vocabulary */
} gto_token_stats;

/* Token-level loss L_token of Eq. 13 (defined in App. B): for every position b the
 * cross-entropy H(p_T, p_M) = -sum_v p_T(v) log p_M(v) from the target's next-token
 * distribution to the draft's under the same teacher-forced prefix, i.e. on the root context
 * rows draft[0,b,0,0,:] and target[0,b,0,:].  With a reduced draft vocabulary p_T is the
 * softmax of the target logits at the mapped ids d2t[0..V_draft) (NULL = identity).  Writes
 * out->loss[b] and grad_root[b,:] = weight * (p_M - p_T), the derivative of weight * H with
 * respect to the draft logits of that row ([B, V_draft], logit dtype, every entry written);
 * a trainer passes weight = 1 / (number of supervised positions).  Needs tree->row_lse from
 * gto_build_tree on the same draft logits.  Any d2t with entries in [0, V_target) is served;
 * an increasing one (a vocabulary subset listed in id order) reads every 32-byte sector of
 * the target row once.  An entry outside the target vocabulary is reported in the device
 * status word (GTO_ERR_BAD_INDEX) and counts as probability 0. */
gto_status gto_token_loss(gto_ctx* ctx, const void* draft_logits, const void* target_logits,
                          const int32_t* d2t, const gto_tree* tree, float weight,
                          void* grad_root, const gto_token_stats* out, void* stream);

/* The total loss of Sec. 3.2, L = L_token + omega * L_GTO, as ONE gradient buffer: the same
 * computation as gto_token_loss, with the root-row gradient weight * (p_M - p_T) of position b
 * going into slice grad[b,0,:] of the buffer gto_group_surrogate_grad filled ([B,D,V_draft]).
 * Step 0 of an accepted path is always taken from the root row, so where that slice already
 * holds a surrogate gradient (path_len[b] > 0 and coeff[b] != 0) the token gradient is added
 * to it, and elsewhere the slice is overwritten.  Afterwards grad[b,0,:] is the derivative of
 * weight * H_b + grad_scale * (sum of the group losses) with respect to the root row of
 * position b, for every b (also where path_row[b,0] is -1).  Call it after
 * gto_group_surrogate_grad on the same stream, with that call's reward and stats. */
gto_status gto_token_loss_accumulate(gto_ctx* ctx, const void* draft_logits,
                                     const void* target_logits, const int32_t* d2t,
                                     const gto_tree* tree, const gto_reward* reward,
                                     const gto_grad_stats* stats, float weight, void* grad,
                                     const gto_token_stats* out, void* stream);

/* SampleGroups of Algorithm 1 under Eq. 6-7: K non-overlapping groups of m adjacent positions
 * of a sequence of length s; start indices are 1-based, 1 <= t_k <= s - m + 1 and
 * t_{k+1} >= t_k + m.  Host-only (no device work): `u` is a HOST array of K uniforms in
 * [0, 1) supplied by the caller, `starts` a HOST array that receives t_1 < ... < t_K.  The
 * paper fixes no law for the draw; this one turns the K uniforms into K independent offsets
 * in [0, s - K m], sorts them and shifts the k-th (0-based) by k m.  Every admissible
 * placement can occur, but not equally often: its weight is the number of orderings of its
 * offsets, so placements with groups packed back to back (equal offsets) are rarer.  Returns
 * GTO_ERR_INVALID_ARG when K*m > s or an argument is out of range. */
gto_status gto_sample_groups(int32_t s, int32_t m, int32_t K, const double* u, int32_t* starts);

/* Synchronises `stream`, then reads and clears the device status word:
 * *host_code = GTO_OK, GTO_ERR_NONFINITE or GTO_ERR_BAD_INDEX.  Kernels check
 * every index they take from a caller's table before using it as an address. */
gto_status gto_device_status(gto_ctx* ctx, void* stream, int32_t* host_code);

/* Number of kernel launches the library has enqueued through this context. */
int64_t gto_launch_count(const gto_ctx* ctx);

/* Kernels of one pass, in launch order (index into the arrays of gto_kernel_times). */
enum {
  GTO_K_DRAFT_ROWS = 0,  /* Sec. 3.1 (i): log-softmax + top-k of every draft row          */
  GTO_K_TREE_BUILD = 1,  /* Sec. 3.1 (i)-(ii): layer-wise expansion, global top-g         */
  GTO_K_REWARD_PLAN = 2, /* list of target rows that are the context of a selected node   */
  GTO_K_TARGET_ROWS = 3, /* Eq. 4: log-sum-exp and greedy token of every listed target row */
  GTO_K_TREE_REWARD = 4, /* Eq. 3-5 and the longest accepted sequence                      */
  GTO_K_GROUP_STATS = 5, /* Eq. 9-12 per group                                             */
  GTO_K_GRAD_ROWS = 6,   /* derivative of Eq. 12 into the draft rows of the accepted path  */
  GTO_K_TOKEN_LOSS = 7,  /* Eq. 13 / App. B: cross-entropy and its gradient on the root rows */
  GTO_K_COUNT = 8
};

/* Per-kernel device timing, off by default.  While enabled, every launch is bracketed by
 * two CUDA events on the caller's stream (host memory only; no device allocation). */
gto_status gto_kernel_timing(gto_ctx* ctx, int enable);

/* Synchronises `stream`, adds up the recorded launches since the last call and clears the
 * record: total_ms[i] = summed device time of kernel i, launches[i] = how many.  Both
 * arrays are HOST arrays of GTO_K_COUNT entries. */
gto_status gto_kernel_times(gto_ctx* ctx, void* stream, double* total_ms, int64_t* launches);

const char* gto_status_string(gto_status s);

#ifdef __cplusplus
}
#endif
#endif /* GTO_H_ */
