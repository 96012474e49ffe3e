// Tree policy G of Sec. 3.1 on the per-row top-k tables: layer-wise expansion (the k best
// of the k*k candidates of each layer by cumulative log-probability become the next
// frontier) and the global top-g prune over all k + (D-1)k^2 candidates.  One warp per
// tree; the rankings are register-resident bitonic networks over 128 (score, index)
// pairs, exchanged with shuffles.  Scores are fp64 sums of (z - lse) so that a ranking
// differs from an exact evaluation only where two scores agree to ~1e-7.
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kE = 4;                  // elements per lane
constexpr int kN = 32 * kE;            // 128 = kMaxLayer = kMaxNodes
constexpr int kWarpsPerCta = 4;
constexpr uint32_t kInvalidAux = 0x7fffffffu;

static_assert(kN == kMaxLayer && kN == kMaxNodes, "network size");

struct Item {
  uint64_t key;  // larger is better
  uint32_t aux;  // smaller is better on equal keys
};

__device__ __forceinline__ bool better(const Item& a, const Item& b) {
  return a.key > b.key || (a.key == b.key && a.aux < b.aux);
}

__device__ __forceinline__ uint64_t score_key(double s) {
  uint64_t u = static_cast<uint64_t>(__double_as_longlong(s + 0.0));
  return u ^ ((u >> 63) ? ~0ull : (1ull << 63));
}
__device__ __forceinline__ double key_score(uint64_t k) {
  uint64_t u = k ^ ((k >> 63) ? (1ull << 63) : ~0ull);
  return __longlong_as_double(static_cast<long long>(u));
}

__device__ __forceinline__ Item shfl_item(const Item& a, int src) {
  Item o;
  o.key = __shfl_sync(kFull, a.key, src);
  o.aux = __shfl_sync(kFull, a.aux, src);
  return o;
}

// One compare-exchange layer of a bitonic network over the blocked layout i = lane*kE + e.
// `desc_mask`: element i sorts descending iff (i & desc_mask) == 0 (0 = all descending).
template <int STRIDE>
__device__ __forceinline__ void bitonic_layer(Item (&x)[kE], int lane, int desc_mask) {
  if constexpr (STRIDE < kE) {
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      if ((e & STRIDE) == 0) {
        int i = lane * kE + e;
        bool desc = (i & desc_mask) == 0;
        Item a = x[e], b = x[e | STRIDE];
        bool a_first = better(a, b);
        bool keep = (a_first == desc);
        x[e] = keep ? a : b;
        x[e | STRIDE] = keep ? b : a;
      }
    }
  } else {
    constexpr int LS = STRIDE / kE;
    bool lower = (lane & LS) == 0;
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      int i = lane * kE + e;
      bool desc = (i & desc_mask) == 0;
      Item o = shfl_item(x[e], lane ^ LS);
      bool mine_better = better(x[e], o);
      bool take_better = (lower == desc);
      x[e] = (mine_better == take_better) ? x[e] : o;
    }
  }
}

template <int SIZE>
__device__ __forceinline__ void bitonic_merge_from(Item (&x)[kE], int lane, int desc_mask) {
  if constexpr (SIZE >= 2) {
    bitonic_layer<SIZE / 2>(x, lane, desc_mask);
    bitonic_merge_from<SIZE / 2>(x, lane, desc_mask);
  }
}

template <int SIZE>
__device__ __forceinline__ void bitonic_sort_upto(Item (&x)[kE], int lane) {
  if constexpr (SIZE >= 2) {
    bitonic_sort_upto<SIZE / 2>(x, lane);
    bitonic_merge_from<SIZE>(x, lane, SIZE == kN ? 0 : SIZE);
  }
}

// Full descending sort of the 128 items held by the warp.
__device__ __forceinline__ void warp_sort_desc(Item (&x)[kE], int lane) {
  bitonic_sort_upto<kN>(x, lane);
}

// a, b sorted descending -> a = the 128 best of the union, sorted descending.
__device__ __forceinline__ void warp_merge_top(Item (&a)[kE], const Item (&b)[kE], int lane) {
#pragma unroll
  for (int e = 0; e < kE; ++e) {
    Item o = shfl_item(b[kE - 1 - e], 31 - lane);  // b reversed
    if (better(o, a[e])) a[e] = o;
  }
  bitonic_merge_from<kN>(a, lane, 0);
}

struct WarpSmem {
  int fpool[kMaxDepth][16];  // fpool[d][j]: pool index of frontier slot j at depth d (1..D-1)
  double fcum[16];           // cumulative score of the current frontier
  double score[kN];
  int sel_pool[kN];
  int parent[kN];
};

__global__ void __launch_bounds__(kWarpsPerCta * 32) tree_build_kernel(TreeBuildArgs a) {
  __shared__ WarpSmem smem[kWarpsPerCta];
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  const int tree = blockIdx.x * kWarpsPerCta + wic;
  if (tree >= a.n_trees) return;
  WarpSmem& sm = smem[wic];
  const int D = a.D, k = a.k, g = a.g, R = a.R, kk = a.k * a.k;
  const double* lse = a.row_lse + static_cast<size_t>(tree) * R;
  const int32_t* top_id = a.top_id + static_cast<size_t>(tree) * R * k;
  const float* top_z = a.top_z + static_cast<size_t>(tree) * R * k;

  // ---- depth 1: the root's k best tokens, already in rank order = pool order
  Item best[kE];  // running global ranking (score desc, pool index asc)
  {
    const double l0 = lse[0];
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      int c = lane * kE + e;
      if (c < k) {
        double sc = static_cast<double>(top_z[c]) - l0;
        best[e].key = score_key(sc);
        best[e].aux = c;
        if (D > 1) {
          sm.fcum[c] = sc;
          sm.fpool[1][c] = c;
        }
      } else {
        best[e].key = 0;
        best[e].aux = kInvalidAux;
      }
    }
  }
  __syncwarp();

  // ---- depths 2..D: k*k candidates per layer
  for (int d = 2; d <= D; ++d) {
    const int base = k + (d - 2) * kk;
    Item cand[kE];
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      int q = lane * kE + e;
      if (q < kk) {
        int j = q / k, c = q - j * k;
        int row = 1 + (d - 2) * k + j;
        double sc = sm.fcum[j] + (static_cast<double>(top_z[row * k + c]) - lse[row]);
        cand[e].key = score_key(sc);
        cand[e].aux = base + q;
      } else {
        cand[e].key = 0;
        cand[e].aux = kInvalidAux;
      }
    }
    __syncwarp();  // all lanes have read fcum
    warp_sort_desc(cand, lane);
    if (d < D) {
#pragma unroll
      for (int e = 0; e < kE; ++e) {
        int rank = lane * kE + e;
        if (rank < k) {
          sm.fcum[rank] = key_score(cand[e].key);
          sm.fpool[d][rank] = static_cast<int>(cand[e].aux);
        }
      }
    }
    warp_merge_top(best, cand, lane);
    __syncwarp();
  }

  // ---- the g best, re-listed in ascending pool index
#pragma unroll
  for (int e = 0; e < kE; ++e) {
    int i = lane * kE + e;
    sm.score[i] = key_score(best[e].key);
    Item it;
    if (i < g) {
      it.key = ~static_cast<uint64_t>(best[e].aux);  // smaller pool index = larger key
      it.aux = i;
    } else {
      it.key = 0;
      it.aux = kInvalidAux;
    }
    best[e] = it;
  }
  __syncwarp();
  warp_sort_desc(best, lane);
  double node_score[kE];
  int node_pool[kE];
#pragma unroll
  for (int e = 0; e < kE; ++e) {
    int n = lane * kE + e;
    if (n < g) {
      node_pool[e] = static_cast<int>(~best[e].key);
      node_score[e] = sm.score[best[e].aux];
      sm.sel_pool[n] = node_pool[e];
    } else {
      node_pool[e] = -1;
      node_score[e] = 0.0;
    }
  }
  __syncwarp();

  // ---- per-node fields
  const size_t obase = static_cast<size_t>(tree) * g;
#pragma unroll
  for (int e = 0; e < kE; ++e) {
    int n = lane * kE + e;
    if (n < g) {
      int p = node_pool[e];
      int depth, c, ctx, par = -1;
      if (p < k) {
        depth = 1;
        c = p;
        ctx = 0;
      } else {
        int dd = (p - k) / kk;
        int q = (p - k) - dd * kk;
        int j = q / k;
        depth = dd + 2;
        c = q - j * k;
        ctx = 1 + dd * k + j;
        int pp = sm.fpool[depth - 1][j];
        int lo = 0, hi = g - 1;  // the parent is selected whenever the child is
        while (lo < hi) {
          int mid = (lo + hi) >> 1;
          if (sm.sel_pool[mid] < pp) lo = mid + 1; else hi = mid;
        }
        par = lo;
      }
      int slot = -1;
      if (depth < D) {
        for (int j = 0; j < k; ++j)
          if (sm.fpool[depth][j] == p) slot = j;
      }
      sm.parent[n] = par;
      a.out.node_token[obase + n] = top_id[ctx * k + c];
      a.out.node_parent[obase + n] = par;
      a.out.node_depth[obase + n] = depth;
      a.out.node_ctx_row[obase + n] = ctx;
      a.out.node_slot[obase + n] = slot;
      a.out.node_pool[obase + n] = p;
      a.out.node_logp[obase + n] =
          static_cast<float>(static_cast<double>(top_z[ctx * k + c]) - lse[ctx]);
      a.out.node_score[obase + n] = node_score[e];
    }
  }
  __syncwarp();

  // ---- ancestor mask: bit a of row n set iff a is n or an ancestor of n
  const int W = (g + 63) / 64;
#pragma unroll
  for (int e = 0; e < kE; ++e) {
    int n = lane * kE + e;
    if (n < g) {
      uint64_t w0 = 0, w1 = 0;
      int x = n;
      for (int step = 0; step <= D && x >= 0; ++step) {
        if (x < 64) w0 |= 1ull << x; else w1 |= 1ull << (x - 64);
        x = sm.parent[x];
      }
      a.out.node_mask[(obase + n) * W] = w0;
      if (W > 1) a.out.node_mask[(obase + n) * W + 1] = w1;
    }
  }
}

}  // namespace

cudaError_t launch_tree_build(const TreeBuildArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.n_trees <= 0) return cudaSuccess;
  dim3 grid((a.n_trees + kWarpsPerCta - 1) / kWarpsPerCta), block(kWarpsPerCta * 32);
  tree_build_kernel<<<grid, block, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
