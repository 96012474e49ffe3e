// Tree policy G of Sec. 3.1 on the per-row top-k tables: layer-wise expansion (the k best
// of the k*k candidates of each layer by cumulative log-probability become the next
// frontier) and the global top-g prune over all k + (D-1)k^2 candidates.  One 128-thread
// CTA per tree, one thread per candidate of a layer.
//
// No sorting network: every ranking is counted.  The k children of one frontier node are
// already in (score descending, index ascending) order, because a row's top-k is and the
// score adds the same parent score to each.  A candidate's rank in its layer is therefore
// its own child index plus, for every other parent, the number of that parent's children
// ahead of it (a binary search over k entries).  The layers are kept sorted in shared
// memory, and a candidate's global rank is its layer rank plus, for every other layer, the
// number of entries ahead of it (a binary search again); only the first g of a layer can
// reach the global top-g.  Ties go to the lower index everywhere: child index within a
// parent, parent slot within a layer, layer (= depth) across layers, i.e. the pool index.
// Scores are fp64 sums of min(z - lse, 0), compared as fp64, so a ranking differs from an exact evaluation only
// where two scores agree to ~1e-7.  The clamp matters: a log-probability is never positive,
// but the fp32-accumulated log-sum-exp of a row with one dominant logit can come out a few
// 1e-7 below that logit; without the clamp such a child would outscore its own parent and
// could be kept by the prune without it.
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kTreeThreads = 128;
static_assert(kMaxLayer <= kTreeThreads, "one thread per layer candidate");
static_assert(kMaxNodes <= kTreeThreads, "one thread per selected node");
constexpr int kMaskWords = kMaxLayer / 32;

// Draft log-probability of a listed token: z - lse, never above 0.
__device__ __forceinline__ double edge_logp(float z, double lse) {
  return fmin(static_cast<double>(z) - lse, 0.0);
}

// The next double above x (x is a score: finite or -inf, never -0 or NaN in a valid tree), so
// that "y > x" can be asked as "y >= next_above(x)".
__device__ __forceinline__ double next_above(double x) {
  const long long b = __double_as_longlong(x);
  return __longlong_as_double(b < 0 ? b - 1 : b + 1);
}

struct TreeSmem {
  double uscore[kMaxLayer];             // scores of the layer in work, by candidate index q
  double fcum[2][kMaxTopK];             // cumulative score of the frontier (double-buffered)
  int fpool[kMaxDepth][kMaxTopK];       // fpool[d][j]: pool index of frontier slot j at depth d
  unsigned selmask[kMaxDepth][kMaskWords];  // selected candidates of each layer, bit q
  int sel_before[kMaxDepth + 1];        // selected nodes in the layers before this one
  int sel_base[kMaxDepth];              // selected candidates of a layer known after the probes
  int sel_count[kMaxDepth];             // selected candidates of a layer
  int parent[kMaxNodes];
};

// Entries of a descending list that come before x; equal scores come before x iff `ties_first`.
// The comparisons are fp64 compares (the fp64 pipe is otherwise idle in this kernel, while a
// 64-bit integer compare costs two instructions on the ALU pipe, which bounds it).
__device__ __forceinline__ int count_ahead(const double* list, int n, double x, bool ties_first) {
  const double bound = ties_first ? x : next_above(x);  // ahead iff y >= bound
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] >= bound) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Same for a list of compile-time length N: a fixed number of branch-free steps (the answer
// is built bit by bit from the top).
template <int N>
__device__ __forceinline__ int count_ahead_fixed(const double* list, double x, bool ties_first) {
  const double bound = ties_first ? x : next_above(x);
  constexpr int kTopBit = N >= 128 ? 128 : N >= 64 ? 64 : N >= 32 ? 32 : N >= 16 ? 16
                          : N >= 8 ? 8 : N >= 4 ? 4 : N >= 2 ? 2 : 1;
  static_assert(N < 256, "step table");
  int pos = 0;  // entries [0, pos) are ahead
#pragma unroll
  for (int step = kTopBit; step > 0; step >>= 1) {
    const int cand = pos + step;
    if (cand <= N && list[cand - 1] >= bound) pos = cand;
  }
  return pos;
}

__device__ __forceinline__ int bits_below(const unsigned (&m)[kMaskWords], int q) {
  int n = 0;
#pragma unroll
  for (int w = 0; w < kMaskWords; ++w) {
    if (w < (q >> 5)) n += __popc(m[w]);
    else if (w == (q >> 5)) n += __popc(m[w] & ((1u << (q & 31)) - 1u));
  }
  return n;
}

template <int K>  // top-k known at compile time, or 0
// 16 resident CTAs per SM (32 registers, no spills): the 2048 trees of the paper's batch are then
// resident at once instead of in two waves of a latency-bound kernel.
__global__ void __launch_bounds__(kTreeThreads, 16) tree_build_kernel(TreeBuildArgs a) {
  extern __shared__ __align__(16) unsigned char dyn[];
  __shared__ TreeSmem sm;
  const int tid = threadIdx.x;
  const int tree = blockIdx.x;
  const int D = a.D, k = K > 0 ? K : a.k, g = a.g, R = a.R, kk = k * k;
  const int P = k + (D - 1) * kk;
  double* skey = reinterpret_cast<double*>(dyn);           // [P] scores of every layer, sorted
  double* lse = skey + P;                                   // [R] staged row log-sum-exps
  float* top_z = reinterpret_cast<float*>(lse + R);        // [R*k] staged top-k logits
  uint8_t* sq = reinterpret_cast<uint8_t*>(top_z + R * k); // [P] candidate index at that rank
  const int32_t* top_id = a.top_id + static_cast<size_t>(tree) * R * k;
  {
    // stage the tree's tables once: the layers then depend on shared memory only
    const double* g_lse = a.row_lse + static_cast<size_t>(tree) * R;
    const float* g_z = a.top_z + static_cast<size_t>(tree) * R * k;
    for (int i = tid; i < R; i += kTreeThreads) lse[i] = g_lse[i];
    for (int i = tid; i < R * k; i += kTreeThreads) top_z[i] = g_z[i];
  }
  auto list_off = [&](int l) { return l == 0 ? 0 : k + (l - 1) * kk; };  // = pool index base
  auto list_len = [&](int l) { return l == 0 ? k : kk; };

  if (tid < D * kMaskWords) (&sm.selmask[0][0])[tid] = 0;
  __syncthreads();
  // ---- depth 1: the root's k best tokens, already in rank order = pool order
  if (tid < k) {
    const double sc = edge_logp(top_z[tid], lse[0]) + 0.0;  // -0 -> +0
    skey[tid] = sc;
    sq[tid] = static_cast<uint8_t>(tid);
    if (D > 1) {
      sm.fcum[0][tid] = sc;
      sm.fpool[1][tid] = tid;
    }
  }
  __syncthreads();

  // ---- depths 2..D: k*k candidates per layer, rank = position in (score desc, q asc) order
  int cur = 0;
  for (int d = 2; d <= D; ++d) {
    const int base = list_off(d - 1);
    const int j = tid / k, c = tid - j * k;
    double sc = 0.0;
    if (tid < kk) {
      const int row = 1 + (d - 2) * k + j;
      sc = sm.fcum[cur][j] + edge_logp(top_z[row * k + c], lse[row]) + 0.0;
      sm.uscore[tid] = sc;
    }
    __syncthreads();
    if (tid < kk) {
      int rank = c;  // the children of one parent are in order already
      if constexpr (K > 0) {
#pragma unroll
        for (int jp = 0; jp < K; ++jp)
          if (jp != j) rank += count_ahead_fixed<K>(&sm.uscore[jp * K], sc, jp < j);
      } else {
        for (int jp = 0; jp < k; ++jp)
          if (jp != j) rank += count_ahead(&sm.uscore[jp * k], k, sc, jp < j);
      }
      skey[base + rank] = sc;
      sq[base + rank] = static_cast<uint8_t>(tid);
      if (d < D && rank < k) {
        sm.fcum[cur ^ 1][rank] = sc;
        sm.fpool[d][rank] = base + tid;
      }
    }
    __syncthreads();
    cur ^= 1;
  }

  // ---- global top-g.  A candidate's rank among all candidates = its rank in its layer +
  //      the entries ahead of it in every other layer, and it grows with the layer rank, so the
  //      selected candidates of a layer are its first s_l.  s_l is found in two rounds instead
  //      of ranking every candidate that could be selected: kProbes evenly spaced layer ranks
  //      bracket it, then the ranks inside the bracket are evaluated.
  auto global_rank = [&](int l, int r) {
    const double x = skey[list_off(l) + r];
    int rank = r;
    if constexpr (K > 0) {
      if (l != 0) rank += count_ahead_fixed<K>(skey, x, true);
      for (int lp = 1; lp < D && rank < g; ++lp)
        if (lp != l) rank += count_ahead_fixed<K * K>(skey + list_off(lp), x, lp < l);
    } else {
      for (int lp = 0; lp < D && rank < g; ++lp)
        if (lp != l) rank += count_ahead(skey + list_off(lp), list_len(lp), x, lp < l);
    }
    return rank;
  };
  constexpr int kProbes = 8;
  static_assert(kMaxDepth * kProbes <= kTreeThreads, "one thread per probe");
  const int cap0 = min(k, g), cap1 = min(kk, g);  // candidates of a layer that can be selected
  const int step0 = (cap0 + kProbes - 1) / kProbes, step1 = (cap1 + kProbes - 1) / kProbes;
  {
    // round 1: probe j of layer l looks at layer rank (j + 1) * step - 1
    const int l = tid / kProbes, j = tid % kProbes;
    bool sel = false;
    if (l < D) {
      const int r = (j + 1) * (l == 0 ? step0 : step1) - 1;
      if (r < (l == 0 ? cap0 : cap1)) sel = global_rank(l, r) < g;
    }
    // the probes of a layer are kProbes neighbouring lanes; the selected ones come first
    const unsigned mine = (__ballot_sync(kFull, sel) >> ((tid & 31) & ~(kProbes - 1))) &
                          ((1u << kProbes) - 1u);
    if (l < D && j == 0) {
      const int base = __popc(mine) * (l == 0 ? step0 : step1);
      sm.sel_base[l] = base;
      sm.sel_count[l] = base;
    }
  }
  __syncthreads();
  {
    // round 2: the layer ranks from the last selected probe up to the next probe
    const int n_items = step0 + (D - 1) * step1;
    for (int t = tid; t < n_items; t += kTreeThreads) {
      const int l = t < step0 ? 0 : 1 + (t - step0) / step1;
      const int i = t < step0 ? t : (t - step0) % step1;
      const int r = sm.sel_base[l] + i;
      if (r < (l == 0 ? cap0 : cap1) && global_rank(l, r) < g) atomicAdd(&sm.sel_count[l], 1);
    }
  }
  __syncthreads();
  if (tid == 0) {
    int n = 0;
    for (int l = 0; l < D; ++l) {
      sm.sel_before[l] = n;
      n += sm.sel_count[l];
    }
    sm.sel_before[D] = n;  // = g
  }
  __syncthreads();
  // one thread per selected candidate: (layer l, layer rank r)
  const int n_sel = sm.sel_before[D];
  int l = 0, r = 0, q = 0;
  const bool mine = tid < n_sel;
  if (mine) {
    while (tid >= sm.sel_before[l + 1]) ++l;
    r = tid - sm.sel_before[l];
    q = sq[list_off(l) + r];
    atomicOr(&sm.selmask[l][q >> 5], 1u << (q & 31));
  }
  __syncthreads();

  // ---- per-node fields, listed in ascending pool index
  const size_t obase = static_cast<size_t>(tree) * g;
  if (mine) {
    const int off = list_off(l);
    const int n = sm.sel_before[l] + bits_below(sm.selmask[l], q);
    const int depth = l + 1;
    int c = q, ctx = 0, par = -1;
    if (l > 0) {
      const int j = q / k;
      c = q - j * k;
      ctx = 1 + (l - 1) * k + j;
      // the parent scores at least as high and has the lower pool index: it is selected too
      const int qp = sm.fpool[l][j] - list_off(l - 1);
      par = sm.sel_before[l - 1] + bits_below(sm.selmask[l - 1], qp);
    }
    sm.parent[n] = par;
    a.out.node_token[obase + n] = top_id[ctx * k + c];
    a.out.node_parent[obase + n] = par;
    a.out.node_depth[obase + n] = depth;
    a.out.node_ctx_row[obase + n] = ctx;
    a.out.node_slot[obase + n] = (depth < D && r < k) ? r : -1;  // frontier slot = layer rank
    a.out.node_pool[obase + n] = off + q;
    a.out.node_logp[obase + n] = static_cast<float>(edge_logp(top_z[ctx * k + c], lse[ctx]));
    a.out.node_score[obase + n] = skey[off + r];
  }
  __syncthreads();

  // ---- ancestor mask: bit a of row n set iff a is n or an ancestor of n
  const int W = (g + 63) / 64;
  if (tid < g) {
    uint64_t w0 = 0, w1 = 0;
    int x = tid;
    for (int step = 0; step <= D && x >= 0; ++step) {
      if (x < 64) w0 |= 1ull << x; else w1 |= 1ull << (x - 64);
      x = sm.parent[x];
    }
    a.out.node_mask[(obase + tid) * W] = w0;
    if (W > 1) a.out.node_mask[(obase + tid) * W + 1] = w1;
  }
}

}  // namespace

cudaError_t launch_tree_build(const TreeBuildArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.n_trees <= 0) return cudaSuccess;
  const int P = a.k + (a.D - 1) * a.k * a.k;
  const int R = 1 + (a.D - 1) * a.k;
  const size_t dyn = static_cast<size_t>(P) * (sizeof(uint64_t) + 1) + R * sizeof(double) +
                     static_cast<size_t>(R) * a.k * sizeof(float);
  if (a.k == 10)
    tree_build_kernel<10><<<a.n_trees, kTreeThreads, dyn, stream>>>(a);  // the paper's top-k
  else
    tree_build_kernel<0><<<a.n_trees, kTreeThreads, dyn, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
