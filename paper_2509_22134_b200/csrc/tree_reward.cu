// Draft Tree Reward (Eq. 3-5) and the longest accepted sequence (Sec. 3.2).
//   reward_plan_kernel : which target rows are the context of a selected node (only
//                        those are streamed), as a compact work list
//   tree_reward_kernel : per tree, p_n = softmax(target row)[token] (the factor of Eq. 4),
//                        path products, L of Eq. 3 per node, the aggregate of Eq. 5 over
//                        the leaves, and for tree 0 the greedy verification walk
// One warp per tree; per-tree arithmetic is fp64 (a few hundred operations).
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kWarpsPerCta = 4;
constexpr int kRowWords = 8;  // bitmap over R <= 256 context rows

__global__ void __launch_bounds__(kWarpsPerCta * 32) reward_plan_kernel(RewardPlanArgs a) {
  __shared__ unsigned flags[kWarpsPerCta][kRowWords];
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  const int tree = blockIdx.x * kWarpsPerCta + wic;
  if (tree >= a.n_trees) return;
  unsigned* fl = flags[wic];
  if (lane < kRowWords) fl[lane] = 0;
  __syncwarp();
  for (int n = lane; n < a.g; n += 32) {
    int r = a.node_ctx_row[static_cast<size_t>(tree) * a.g + n];
    if (r < 0 || r >= a.R) {  // not a row of this tree: report, do not touch memory with it
      atomicOr(a.status, kStatusBadIndex);
      continue;
    }
    atomicOr(&fl[r >> 5], 1u << (r & 31));
  }
  __syncwarp();
  int total = 0;
#pragma unroll
  for (int w = 0; w < kRowWords; ++w) total += __popc(fl[w]);
  int base = 0;
  if (lane == 0) base = atomicAdd(a.list_count, total);
  base = __shfl_sync(kFull, base, 0);
  for (int r = lane; r < a.R; r += 32) {
    unsigned word = fl[r >> 5];
    size_t gid = static_cast<size_t>(tree) * a.R + r;
    if (word & (1u << (r & 31))) {
      int rank = __popc(word & ((1u << (r & 31)) - 1));
      for (int w = 0; w < (r >> 5); ++w) rank += __popc(fl[w]);
      a.list[base + rank] = static_cast<int32_t>(gid);
    } else {
      a.row_lse_t[gid] = __longlong_as_double(0x7ff8000000000000ll);
      a.row_argmax_t[gid] = -1;
    }
  }
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
__device__ __forceinline__ double warp_max_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
  return v;
}

struct RewardSmem {
  double p[kMaxNodes];
  double Pp[kMaxNodes];
  double Lc[kMaxNodes];
  int parent[kMaxNodes];
  int tok_t[kMaxNodes];
  int depth[kMaxNodes];
  int has_child[kMaxNodes];
};

template <typename T>
__global__ void __launch_bounds__(kWarpsPerCta * 32) tree_reward_kernel(RewardArgs a) {
  __shared__ RewardSmem smem[kWarpsPerCta];
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  const int tree = blockIdx.x * kWarpsPerCta + wic;
  if (tree >= a.G * a.B) return;
  RewardSmem& sm = smem[wic];
  const int g = a.g, R = a.R, D = a.D, k = a.k;
  const size_t nb = static_cast<size_t>(tree) * g;
  const size_t rb = static_cast<size_t>(tree) * R;
  const char* tbase = static_cast<const char*>(a.target);

  // ---- target probability of every node's token in its context (Eq. 4 factor)
  for (int n = lane; n < g; n += 32) {
    const int ctx = a.tree.node_ctx_row[nb + n];
    const int tok = a.tree.node_token[nb + n];
    const int par = a.tree.node_parent[nb + n];
    const int dep = a.tree.node_depth[nb + n];
    // every index is checked before it addresses anything
    bool ok = ctx >= 0 && ctx < R && tok >= 0 && tok < a.V_draft && par >= -1 && par < n &&
              dep >= 1 && dep <= D;
    int tt = -1;
    if (ok) {
      tt = a.d2t ? a.d2t[tok] : tok;
      ok = tt >= 0 && tt < a.V_target;
    }
    double pr = 0.0;
    if (ok) {
      const float z = T::load1(tbase, (rb + ctx) * static_cast<size_t>(a.V_target) + tt);
      pr = exp(static_cast<double>(z) - a.out.row_lse_t[rb + ctx]);
    } else {
      atomicOr(a.status, kStatusBadIndex);
    }
    sm.p[n] = pr;
    sm.parent[n] = ok ? par : -1;
    sm.depth[n] = ok ? dep : 1;
    sm.tok_t[n] = ok ? tt : -1;
    sm.has_child[n] = 0;
  }
  __syncwarp();
  for (int n = lane; n < g; n += 32)
    if (sm.parent[n] >= 0) sm.has_child[sm.parent[n]] = 1;
  // ---- Eq. 4 path products and Eq. 3 partial sums, one depth level at a time
  for (int d = 1; d <= D; ++d) {
    for (int n = lane; n < g; n += 32) {
      if (sm.depth[n] == d) {
        int par = sm.parent[n];
        double pp = sm.p[n] * (par < 0 ? 1.0 : sm.Pp[par]);
        sm.Pp[n] = pp;
        sm.Lc[n] = (par < 0 ? 0.0 : sm.Lc[par]) + pp;
      }
    }
    __syncwarp();
  }
  // ---- Eq. 5 over the leaves
  const double eta = static_cast<double>(a.eta);
  const bool all_nodes = (a.flags & GTO_FLAG_SEQ_ALL_NODES) != 0;  // every node ends a sequence
  double mx = -INFINITY, sumL = 0.0, sumPp = 0.0;
  int leaves = 0;
  for (int n = lane; n < g; n += 32) {
    sumPp += sm.Pp[n];
    if (all_nodes || !sm.has_child[n]) {
      ++leaves;
      mx = fmax(mx, sm.Lc[n]);
      sumL += sm.Lc[n];
    }
  }
  mx = warp_max_f64(mx);
  sumL = warp_sum_f64(sumL);
  sumPp = warp_sum_f64(sumPp);
  leaves = __reduce_add_sync(kFull, leaves);
  double reward;
  if (a.agg == GTO_AGG_MAX) {
    reward = mx;
  } else if (a.agg == GTO_AGG_MEAN) {
    reward = sumL / leaves;
  } else {
    double se = 0.0;
    for (int n = lane; n < g; n += 32)
      if (all_nodes || !sm.has_child[n]) se += exp(eta * (sm.Lc[n] - mx));
    se = warp_sum_f64(se);
    reward = (eta * mx + log(se)) / eta;
  }
  if (lane == 0) {
    a.out.reward[tree] = reward;
    a.out.etree[tree] = sumPp;
    a.out.n_leaves[tree] = leaves;
  }
  for (int n = lane; n < g; n += 32) {
    a.out.node_ptarget[nb + n] = static_cast<float>(sm.p[n]);
    a.out.node_pathprod[nb + n] = static_cast<float>(sm.Pp[n]);
    a.out.node_L[nb + n] = static_cast<float>(sm.Lc[n]);
  }

  // ---- longest accepted sequence of the current draft's tree (t = 0): follow the greedy
  //      target token through the selected children
  if (tree < a.B && (a.flags & GTO_FLAG_PATH_MAX_EXPECTED)) {
    // the other reading: the sequence with the largest L (Eq. 3), lowest list position on
    // ties, taken whole from the root to its last node
    const int b = tree;
    double best = -INFINITY;
    int at = g;
    for (int n = lane; n < g; n += 32)
      if ((all_nodes || !sm.has_child[n]) && sm.Lc[n] > best) {
        best = sm.Lc[n];
        at = n;
      }
    const double top = warp_max_f64(best);
    at = __reduce_min_sync(kFull, best == top ? at : g);
    int len = 0;
    if (at < g) {
      len = sm.depth[at];
      int n = at;
      for (int j = len - 1; j >= 0 && n >= 0; --j) {  // every lane walks the same chain
        if (lane == 0) {
          a.out.path_node[b * D + j] = n;
          a.out.path_row[b * D + j] = a.tree.node_ctx_row[nb + n];
          a.out.path_token[b * D + j] = a.tree.node_token[nb + n];
          a.out.path_logp[b * D + j] = a.tree.node_logp[nb + n];
        }
        n = sm.parent[n];
      }
    }
    if (lane == 0) a.out.path_len[b] = len;
    for (int j = len + lane; j < D; j += 32) {
      a.out.path_node[b * D + j] = -1;
      a.out.path_row[b * D + j] = -1;
      a.out.path_token[b * D + j] = -1;
      a.out.path_logp[b * D + j] = 0.f;
    }
  } else if (tree < a.B) {
    const int b = tree;
    int cur = -1, row = 0, len = 0;
    while (len < D) {
      int am = a.out.row_argmax_t[rb + row];
      int found = -1;
      for (int n0 = 0; n0 < g; n0 += 32) {
        int n = n0 + lane;
        bool hit = n < g && sm.parent[n] == cur && sm.tok_t[n] == am;
        unsigned bal = __ballot_sync(kFull, hit);
        if (bal && found < 0) found = n0 + __ffs(bal) - 1;
      }
      if (found < 0) break;
      if (lane == 0) {
        a.out.path_node[b * D + len] = found;
        a.out.path_row[b * D + len] = row;
        a.out.path_token[b * D + len] = a.tree.node_token[nb + found];
        a.out.path_logp[b * D + len] = a.tree.node_logp[nb + found];
      }
      ++len;
      int slot = a.tree.node_slot[nb + found];
      int depth = sm.depth[found];
      if (slot < 0 || depth >= D) break;
      if (slot >= k) {  // not a frontier slot: report and stop the walk
        if (lane == 0) atomicOr(a.status, kStatusBadIndex);
        break;
      }
      cur = found;
      row = 1 + (depth - 1) * k + slot;
    }
    if (lane == 0) a.out.path_len[b] = len;
    for (int j = len + lane; j < D; j += 32) {
      a.out.path_node[b * D + j] = -1;
      a.out.path_row[b * D + j] = -1;
      a.out.path_token[b * D + j] = -1;
      a.out.path_logp[b * D + j] = 0.f;
    }
  }
}

}  // namespace

cudaError_t launch_reward_plan(const RewardPlanArgs& a, cudaStream_t stream, int64_t* launches) {
  cudaError_t e = cudaMemsetAsync(a.list_count, 0, sizeof(int32_t), stream);
  if (e != cudaSuccess) return e;
  dim3 grid((a.n_trees + kWarpsPerCta - 1) / kWarpsPerCta), block(kWarpsPerCta * 32);
  reward_plan_kernel<<<grid, block, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_tree_reward(const RewardArgs& a, cudaStream_t stream, int64_t* launches) {
  int n_trees = a.G * a.B;
  dim3 grid((n_trees + kWarpsPerCta - 1) / kWarpsPerCta), block(kWarpsPerCta * 32);
  if (a.dtype == GTO_BF16)
    tree_reward_kernel<Bf16><<<grid, block, 0, stream>>>(a);
  else if (a.dtype == GTO_F16)
    tree_reward_kernel<F16><<<grid, block, 0, stream>>>(a);
  else
    tree_reward_kernel<F32><<<grid, block, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
