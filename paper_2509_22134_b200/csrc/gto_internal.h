// Host-side declarations shared by the GTO translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gto.h"

namespace gto {

inline int elem_bytes(int dtype) { return dtype == GTO_F32 ? 4 : 2; }
inline bool valid_dtype(int dtype) { return dtype == GTO_F32 || dtype == GTO_BF16 || dtype == GTO_F16; }

constexpr int kMaxTopK = 16;       // per-row top-k the row kernel can hold
constexpr int kMaxLayer = 128;     // k*k candidates per layer
constexpr int kMaxNodes = 128;     // g
constexpr int kMaxDepth = 16;      // D

// One pass over logit rows: log-sum-exp and the top-k (value desc, id asc) of each row.
struct RowReduceArgs {
  const void* logits;        // tensor base
  int dtype;                 // gto_dtype
  int V;                     // row length
  int R;                     // context rows per tree
  int pad;                   // unused rows between row 0 and row 1 of a tree in the tensor
  const int32_t* list;       // optional: global row ids (tree*R + r) to process
  const int32_t* list_count; // device count of entries in list (with list)
  int n_rows;                // rows to process (upper bound on the list length with list)
  int k;                     // top-k per row
  double* out_lse;           // [trees*R]
  int32_t* out_id;           // [trees*R, k]
  float* out_z;              // [trees*R, k] or null
  int32_t* status;           // device status word
  int grid_cap;              // with list: most CTAs to launch (0 = one per possible entry)
  int split_below;           // at most this many rows: split each row over a cluster (0 = never)
  int sms;                   // multiprocessors of the device (0 = unknown)
};
cudaError_t launch_row_reduce(const RowReduceArgs& a, cudaStream_t stream, int64_t* launches);

struct TreeBuildArgs {
  int n_trees, D, k, g, R;
  const double* row_lse;   // [trees*R]
  const int32_t* top_id;   // [trees*R, k]
  const float* top_z;      // [trees*R, k]
  gto_tree out;
};
cudaError_t launch_tree_build(const TreeBuildArgs& a, cudaStream_t stream, int64_t* launches);

struct RewardPlanArgs {
  int n_trees, g, R;
  const int32_t* node_ctx_row;  // [trees, g]
  int32_t* list;                // [trees*R] out: needed global row ids
  int32_t* list_count;          // out (zeroed by the launcher)
  double* row_lse_t;            // [trees*R] poisoned to NaN for rows not needed
  int32_t* row_argmax_t;        // [trees*R] set to -1 likewise
  int32_t* status;              // device status word
};
cudaError_t launch_reward_plan(const RewardPlanArgs& a, cudaStream_t stream, int64_t* launches);

struct RewardArgs {
  int B, G, D, k, g, R, V_draft, V_target, dtype, agg;
  uint32_t flags;
  int32_t* status;
  float eta;
  const void* target;
  const int32_t* d2t;
  gto_tree tree;
  gto_reward out;
};
cudaError_t launch_tree_reward(const RewardArgs& a, cudaStream_t stream, int64_t* launches);

struct GradArgs {
  int B, D, k, R, m, V, dtype;
  float clip_eps, std_delta, grad_scale;
  uint32_t flags;
  const void* draft;
  const double* row_lse;  // [G*B*R] draft lse (tree 0 rows are used)
  gto_reward reward;
  const float* old_logp;
  void* grad;
  gto_grad_stats out;
  int32_t* status;
  int32_t* live_list;   // with GTO_FLAG_GRAD_LIVE_ROWS: workspace [B*D], the slices b*D + j that
  int32_t* live_count;  //   carry a gradient and their number; null otherwise
  int live_grid;        // CTAs that walk the list
};
struct TokenLossArgs {
  int B, k, R, V_draft, V_target, dtype;
  float weight;
  const void* draft;       // [G,B,D,k,V_draft]; row [0,b,0,0,:] is read
  const void* target;      // [G,B,R,V_target]; row [0,b,0,:] is read
  const int32_t* d2t;      // [V_draft] or null (identity)
  const double* row_lse;   // [G*B*R] draft log-sum-exp (entry of row 0 of tree (0,b))
  void* grad_out;          // gradient rows in the logit dtype: row b starts at b * out_stride
  int64_t out_stride;      // elements between the rows of consecutive positions
  const int32_t* acc_path_len;  // accumulate mode: [B] accepted lengths, else null
  const double* acc_coeff;      // accumulate mode: [B] surrogate coefficients
  double* loss;            // [B]
  double* lse_t;           // [B]
  int32_t* status;
};
cudaError_t launch_token_loss(const TokenLossArgs& a, int sms, cudaStream_t stream,
                              int64_t* launches);

cudaError_t launch_group_stats(const GradArgs& a, cudaStream_t stream, int64_t* launches);
cudaError_t launch_grad_rows(const GradArgs& a, cudaStream_t stream, int64_t* launches);

}  // namespace gto
