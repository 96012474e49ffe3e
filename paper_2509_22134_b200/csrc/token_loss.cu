// Token-level loss of Eq. 13 / App. B: for every position the cross-entropy
// H(p_T, p_M) = -sum_v p_T(v) log p_M(v) between the target's and the draft's next-token
// distributions under the same teacher-forced prefix (the root context row of the current
// draft's tree), and its derivative weight * (p_M - p_T) with respect to the draft logits.
// With a reduced draft vocabulary the target distribution is the softmax of the target
// logits at the mapped ids.
//
// Streaming kernel (token_loss_stream_kernel): a position is shared by a thread-block
// cluster; every CTA owns a contiguous range of draft ids.  Pass A streams the CTA's part of
// the target row with 16-byte loads, keeps the logits of the mapped ids in shared memory in
// draft-id order and sums their exponentials; the cluster then combines the partial sums
// through distributed shared memory.  Pass B streams the draft row once, takes the target
// logits from shared memory, and writes the gradient row.  Every byte of the two rows is read
// once from HBM and nothing is gathered.  With an id map this needs the map to be increasing
// (a vocabulary subset listed in id order): then the mapped target logits, taken in target-id
// order, are already in draft-id order, and "is this target id mapped, and to which draft id"
// is a bit test and a prefix pop-count over a bitmap of the map's image (token_map_*
// kernels, rebuilt on every call because the map is the caller's).  A map that is injective
// but not increasing is detected while the bitmap is built and handled by the gathering
// kernel below instead.
//
// Gathering kernel (token_loss_gather_kernel): one CTA per position, two passes over the two
// rows (the second hits L2); the id-map gather is laid out so that a warp load touches few
// 32-byte sectors.  Serves any injective map and rows too long for the cluster's shared memory.
#include <cooperative_groups.h>

#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

namespace cg = cooperative_groups;

#ifndef GTO_TOK_THREADS
#define GTO_TOK_THREADS 256
#endif
constexpr int kTokThreads = GTO_TOK_THREADS;
constexpr int kTokWarps = kTokThreads / 32;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// ------------------------------------------------------------------ bitmap of the id map
// One CTA builds, for the call's id map: bitmap[w] bit i = target id 32 w + i is the image of a
// draft id; prefix[w] = number of mapped target ids below 32 w; map_state[0] = 1 if the map is
// not strictly increasing or holds an id outside the target vocabulary (the streaming kernel
// then leaves the call to the gathering kernel).  A few thousand words: one launch is cheaper
// than a grid-wide version with its extra launches.
__global__ void __launch_bounds__(1024) token_map_build_kernel(
    const int32_t* __restrict__ d2t, int V_draft, int V_target, int n_words, uint32_t* bitmap,
    uint32_t* __restrict__ prefix, int32_t* map_state, int32_t* __restrict__ status) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int w = tid; w < n_words; w += 1024) bitmap[w] = 0;
  if (tid == 0) {
    carry = 0;
    map_state[0] = 0;
  }
  __syncthreads();
  for (int v = tid; v < V_draft; v += 1024) {
    const int id = d2t[v];
    if (id < 0 || id >= V_target) {
      atomicOr(status, kStatusBadIndex);
      atomicOr(map_state, 1);  // ranks would no longer be draft ids
      continue;
    }
    if (v > 0 && d2t[v - 1] >= id) atomicOr(map_state, 1);
    atomicOr(bitmap + (id >> 5), 1u << (id & 31));
  }
  __syncthreads();
  for (int base = 0; base < n_words; base += 1024) {
    const int w = base + tid;
    const uint32_t c = w < n_words ? __popc(bitmap[w]) : 0u;
    uint32_t inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t up = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += up;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t before = carry;
    for (int q = 0; q < warp; ++q) before += warp_tot[q];
    if (w < n_words) prefix[w] = before + inc - c;
    __syncthreads();
    if (tid == 1023) carry = before + inc;
    __syncthreads();
  }
}

// ------------------------------------------------------------------ streaming kernel
struct TokPartial {
  float m;     // largest mapped target logit of the CTA's range (-inf if none)
  double s;    // sum of exp(t - m) over the range
  double h;    // the range's part of sum p_T log p_M
};

template <typename T>
__global__ void __launch_bounds__(kTokThreads) token_loss_stream_kernel(TokenLossArgs a) {
  constexpr int E = T::kPerVec;
  extern __shared__ __align__(16) unsigned char s_raw[];  // the range's target logits, logit dtype
  __shared__ TokPartial part;
  __shared__ float s_m[kTokWarps];
  __shared__ double s_s[kTokWarps];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = static_cast<int>(cluster.num_blocks());
  const int c = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // the map turned out not to be increasing: the gathering kernel does this call
  if (a.d2t != nullptr && a.map_state[0] != 0) return;

  const int nvec = a.V_draft / E;
  const int per = (nvec + C - 1) / C;
  const int vec0 = min(c * per, nvec), vec1 = min(vec0 + per, nvec);  // the CTA's draft vectors
  const int id0 = vec0 * E, id1 = vec1 * E;                           // its draft ids
  const char* zd = static_cast<const char*>(a.draft) +
                   tensor_row(b, 0, a.R, a.k - 1) * a.V_draft * T::kBytes;
  const char* zt = static_cast<const char*>(a.target) +
                   static_cast<int64_t>(b) * a.R * a.V_target * T::kBytes;
  using Elem = typename T::Storage;
  Elem* s_t = reinterpret_cast<Elem*>(s_raw);

  // ---- pass A: the range's mapped target logits into shared memory, then their max and sum
  float m = -INFINITY, s = 0.f;
  auto take = [&](const float (&t)[E]) {
    float vmax = t[0];
#pragma unroll
    for (int e = 1; e < E; ++e) vmax = fmaxf(vmax, t[e]);
    if (vmax > m) {
      s *= ex2_approx((m - vmax) * kLog2e);
      m = vmax;
    }
    if (m != -INFINITY) {
#pragma unroll
      for (int e = 0; e < E; ++e) s += ex2_approx((t[e] - m) * kLog2e);
    }
  };
  if (a.d2t == nullptr) {
    for (int i = vec0 + tid; i < vec1; i += kTokThreads) {
      reinterpret_cast<uint4*>(s_raw)[i - vec0] = ld_stream16(zt + static_cast<size_t>(i) * 16);
    }
  } else if (id1 > id0) {
    const int t_lo = a.d2t[id0], t_hi = a.d2t[id1 - 1];  // target ids of the range's ends
    const int i_end = t_hi / E + 1;
    constexpr int U = 4;  // vectors in flight per thread
    for (int i0 = t_lo / E + tid; i0 < i_end; i0 += U * kTokThreads) {
      uint4 v[U];
      uint32_t word[U], pre[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * kTokThreads;
        if (i < i_end) {
          v[u] = ld_stream16(zt + static_cast<size_t>(i) * 16);
          word[u] = __ldg(a.map_bits + ((i * E) >> 5));
          pre[u] = __ldg(a.map_prefix + ((i * E) >> 5));
        } else {
          word[u] = 0;
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        // E consecutive target ids: their bits of the image bitmap, and the draft id (rank)
        // of the first mapped one among them
        const int first = (i0 + u * kTokThreads) * E;
        const unsigned bits = (word[u] >> (first & 31)) & ((1u << E) - 1u);
        unsigned todo = bits;
        int rank = static_cast<int>(pre[u]) + __popc(word[u] & ((1u << (first & 31)) - 1u));
        while (todo) {  // about E * V_draft / V_target mapped ids per vector
          const int e = __ffs(todo) - 1;
          todo &= todo - 1;
          // neighbouring ranges share their end vectors: keep the ids of this range only
          if (rank >= id0 && rank < id1) s_t[rank - id0] = T::element(v[u], e);
          ++rank;
        }
      }
    }
  }
  __syncthreads();
  // the range's log-sum-exp from shared memory (dense, in draft-id order)
  for (int i = tid; i < vec1 - vec0; i += kTokThreads) {
    float t[E];
    T::unpack(reinterpret_cast<const uint4*>(s_raw)[i], t);
    take(t);
  }
  {
    const float wm = warp_max_f32(m);
    const double ws =
        warp_sum_f64(m == -INFINITY ? 0.0 : static_cast<double>(s * ex2_approx((m - wm) * kLog2e)));
    if (lane == 0) {
      s_m[warp] = wm;
      s_s[warp] = ws;
    }
  }
  __syncthreads();
  if (tid == 0) {
    float M = s_m[0];
    for (int w = 1; w < kTokWarps; ++w) M = fmaxf(M, s_m[w]);
    double S = 0.0;
    for (int w = 0; w < kTokWarps; ++w)
      if (s_m[w] != -INFINITY) S += s_s[w] * exp2(static_cast<double>((s_m[w] - M) * kLog2e));
    part.m = M;
    part.s = S;
  }
  cluster.sync();  // every range's partial sum is visible; s_t is complete
  double lse;
  {
    float M = -INFINITY;
    for (int q = 0; q < C; ++q) M = fmaxf(M, cluster.map_shared_rank(&part, q)->m);
    double S = 0.0;
    for (int q = 0; q < C; ++q) {
      const TokPartial* pq = cluster.map_shared_rank(&part, q);
      if (pq->m != -INFINITY) S += pq->s * exp2(static_cast<double>((pq->m - M) * kLog2e));
    }
    lse = static_cast<double>(M) + log(S);
  }
  if (c == 0 && tid == 0) {
    a.lse_t[b] = lse;
    if (!isfinite(lse)) atomicOr(a.status, kStatusNonFinite);
  }
  const float lse_t = static_cast<float>(lse);
  const float lse_d = static_cast<float>(a.row_lse[static_cast<size_t>(b) * a.R]);

  // ---- pass B: loss and gradient of the CTA's draft ids
  char* out = static_cast<char*>(a.grad_out) + static_cast<size_t>(b) * a.out_stride * T::kBytes;
  // with `accumulate` the row may already hold the surrogate's gradient of the same draft row
  const bool add = a.acc_path_len != nullptr && a.acc_path_len[b] > 0 && a.acc_coeff[b] != 0.0;
  float h = 0.f;
  for (int i = vec0 + tid; i < vec1; i += kTokThreads) {
    float t[E], z[E], g[E];
    T::unpack(reinterpret_cast<const uint4*>(s_raw)[i - vec0], t);
    T::unpack(ld_stream16(zd + static_cast<size_t>(i) * 16), z);
    if (add) {
      T::unpack(*reinterpret_cast<const uint4*>(out + static_cast<size_t>(i) * 16), g);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) g[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const float lq = z[e] - lse_d;                          // log p_M
      const float pt = ex2_approx((t[e] - lse_t) * kLog2e);  // p_T
      h = fmaf(pt, lq, h);
      g[e] = fmaf(a.weight, ex2_approx(lq * kLog2e) - pt, g[e]);
    }
    st_stream16(out + static_cast<size_t>(i) * 16, T::pack(g));
  }
  const double hs = warp_sum_f64(static_cast<double>(h));
  __syncthreads();  // s_s is reused
  if (lane == 0) s_s[warp] = hs;
  __syncthreads();
  if (tid == 0) {
    double H = 0.0;
    for (int w = 0; w < kTokWarps; ++w) H += s_s[w];
    part.h = H;
  }
  cluster.sync();  // the partial losses are visible; nobody has left while its partials were read
  if (c == 0 && tid == 0) {
    double H = 0.0;
    for (int q = 0; q < C; ++q) H += cluster.map_shared_rank(&part, q)->h;
    a.loss[b] = -H;
  }
  cluster.sync();  // the first CTA has read every partial before any CTA exits
}

// ------------------------------------------------------------------ gathering kernel
template <typename T>
__global__ void __launch_bounds__(kTokThreads, 8) token_loss_gather_kernel(TokenLossArgs a) {
  constexpr int E = T::kPerVec;
  constexpr int kChunk = 32 * E;  // draft ids a warp handles at a time
  __shared__ float s_max[kTokWarps];
  __shared__ double s_sum[kTokWarps];
  __shared__ double s_lse;
  __shared__ __align__(16) float s_t[kTokWarps][kChunk];  // a warp's gathered target logits
  // an increasing map is served by the streaming kernel of the same call
  if (a.map_state != nullptr && a.map_state[0] == 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  const char* zd = static_cast<const char*>(a.draft) +
                   tensor_row(b, 0, a.R, a.k - 1) * a.V_draft * T::kBytes;
  const char* zt = static_cast<const char*>(a.target) +
                   static_cast<int64_t>(b) * a.R * a.V_target * T::kBytes;
  const int nvec = a.V_draft / E;
  const int nchunk = (nvec + 31) / 32;

  // Target logits of the chunk's draft ids.  With an id map, lane l takes ids
  // chunk*kChunk + e*32 + l: 32 neighbouring draft ids map to target ids a few apart, so one
  // warp load touches a handful of 32-byte sectors instead of 32.  Missing ids read -inf.
  auto gather_strided = [&](int chunk, float (&t)[E]) {
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const int v = chunk * kChunk + e * 32 + lane;
      t[e] = -INFINITY;
      if (v < a.V_draft) {
        const int id = __ldg(a.d2t + v);
        if (id >= 0 && id < a.V_target) t[e] = T::load1(zt, id);
        else atomicOr(a.status, kStatusBadIndex);  // reported; the id counts as probability 0
      }
    }
  };
  // Without a map: the lane's own 16-byte vector (ids chunk*kChunk + l*E ...).
  auto load_direct = [&](int chunk, float (&t)[E]) {
    const int i = chunk * 32 + lane;
    if (i < nvec) {
      T::unpack(ld_stream16(zt + static_cast<size_t>(i) * 16), t);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) t[e] = -INFINITY;
    }
  };

  // ---- pass A: log-sum-exp of the mapped target logits (running maximum per thread)
  float m = -INFINITY, s = 0.f;
  for (int c = warp; c < nchunk; c += kTokWarps) {
    float t[E];
    if (a.d2t != nullptr) gather_strided(c, t); else load_direct(c, t);
    float vmax = t[0];
#pragma unroll
    for (int e = 1; e < E; ++e) vmax = fmaxf(vmax, t[e]);
    if (vmax > m) {
      s *= ex2_approx((m - vmax) * kLog2e);
      m = vmax;
    }
    if (m != -INFINITY) {
#pragma unroll
      for (int e = 0; e < E; ++e) s += ex2_approx((t[e] - m) * kLog2e);
    }
  }
  {
    const float wm = warp_max_f32(m);
    const double part =
        warp_sum_f64(m == -INFINITY ? 0.0 : static_cast<double>(s * ex2_approx((m - wm) * kLog2e)));
    if (lane == 0) {
      s_max[warp] = wm;
      s_sum[warp] = part;
    }
  }
  __syncthreads();
  if (tid == 0) {
    float M = s_max[0];
    for (int w = 1; w < kTokWarps; ++w) M = fmaxf(M, s_max[w]);
    double S = 0.0;
    for (int w = 0; w < kTokWarps; ++w)
      if (s_max[w] != -INFINITY)
        S += s_sum[w] * exp2(static_cast<double>((s_max[w] - M) * kLog2e));
    const double lse = static_cast<double>(M) + log(S);
    s_lse = lse;
    a.lse_t[b] = lse;
    if (!isfinite(lse)) atomicOr(a.status, kStatusNonFinite);
  }
  __syncthreads();
  const float lse_t = static_cast<float>(s_lse);
  const float lse_d = static_cast<float>(a.row_lse[static_cast<size_t>(b) * a.R]);

  // ---- pass B: loss and gradient; lane l owns the vector of ids chunk*kChunk + l*E ...
  char* out = static_cast<char*>(a.grad_out) + static_cast<size_t>(b) * a.out_stride * T::kBytes;
  const bool add = a.acc_path_len != nullptr && a.acc_path_len[b] > 0 && a.acc_coeff[b] != 0.0;
  float h = 0.f;
  for (int c = warp; c < nchunk; c += kTokWarps) {
    float t[E], z[E], g[E];
    if (a.d2t != nullptr) {
      // gather in the sector-friendly order, then hand each lane its own E values
      gather_strided(c, t);
      __syncwarp();
#pragma unroll
      for (int e = 0; e < E; ++e) s_t[warp][e * 32 + lane] = t[e];
      __syncwarp();
#pragma unroll
      for (int e = 0; e < E; ++e) t[e] = s_t[warp][lane * E + e];
    } else {
      load_direct(c, t);
    }
    const int i = c * 32 + lane;
    if (i < nvec) {
      T::unpack(ld_stream16(zd + static_cast<size_t>(i) * 16), z);
      if (add) {
        T::unpack(*reinterpret_cast<const uint4*>(out + static_cast<size_t>(i) * 16), g);
      } else {
#pragma unroll
        for (int e = 0; e < E; ++e) g[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < E; ++e) {
        const float lq = z[e] - lse_d;                               // log p_M
        const float pt = ex2_approx((t[e] - lse_t) * kLog2e);       // p_T
        h = fmaf(pt, lq, h);
        g[e] = fmaf(a.weight, ex2_approx(lq * kLog2e) - pt, g[e]);
      }
      st_stream16(out + static_cast<size_t>(i) * 16, T::pack(g));
    }
  }
  double hs = warp_sum_f64(static_cast<double>(h));
  __syncthreads();  // s_sum is reused
  if (lane == 0) s_sum[warp] = hs;
  __syncthreads();
  if (tid == 0) {
    double H = 0.0;
    for (int w = 0; w < kTokWarps; ++w) H += s_sum[w];
    a.loss[b] = -H;
  }
}

template <typename T>
cudaError_t launch_stream(const TokenLossArgs& a, int C, size_t smem, cudaStream_t stream) {
  // raise the kernel's dynamic shared memory limit when a call needs more than any before it
  // (per device: the attribute belongs to the device's copy of the function)
  static int allowed[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || static_cast<int>(smem) > allowed[dev]) {
    e = cudaFuncSetAttribute(token_loss_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) allowed[dev] = static_cast<int>(smem);
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(a.B) * C);
  cfg.blockDim = dim3(kTokThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = C;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, token_loss_stream_kernel<T>, a);
}

}  // namespace

// CTAs per position for the streaming kernel, from timings on B200 (us per call, B = 1024,
// bf16): with an id map 32 000 -> 128 256, 2 CTAs per position are fastest; without a map the
// gathering kernel (target re-read from L2) wins while a row is short (54 vs 67 at 32 000 ids)
// and 4 CTAs win on long rows (155 vs 179 at 151 936 ids).  Small batches take the largest
// portable cluster so that the device fills.  0 = use the gathering kernel.
int token_loss_cluster_size(int B, int V_draft, bool mapped, int dtype, int sms) {
#ifdef GTO_TOK_CLUSTER
  return GTO_TOK_CLUSTER;  // tuning builds
#endif
  const size_t row = static_cast<size_t>(V_draft) * elem_bytes(dtype);
  if (!mapped && row < 128 * 1024 && B >= sms) return 0;
  int C = mapped ? 2 : 4;
  while (C < 8 && static_cast<int64_t>(B) * C < 2ll * sms) C *= 2;  // a small batch
  while (C < 8 && (row + C - 1) / C + 64 > 96 * 1024) C *= 2;        // a CTA's share must fit
  return (row + C - 1) / C + 64 <= 200 * 1024 ? C : 0;
}

cudaError_t launch_token_loss(const TokenLossArgs& a, int sms, cudaStream_t stream,
                              int64_t* launches) {
  if (a.B <= 0) return cudaSuccess;
  const int C = token_loss_cluster_size(a.B, a.V_draft, a.d2t != nullptr, a.dtype, sms);
  cudaError_t e = cudaSuccess;
  if (C > 0 && a.d2t != nullptr) {
    // the bitmap of the map's image and its prefix counts
    const int n_words = (a.V_target + 31) / 32 + 1;
    token_map_build_kernel<<<1, 1024, 0, stream>>>(a.d2t, a.V_draft, a.V_target, n_words, a.map_bits,
                                                   a.map_prefix, a.map_state, a.status);
    ++*launches;
  }
  if (C > 0) {
    const int E = 16 / elem_bytes(a.dtype);
    const int per = (a.V_draft / E + C - 1) / C;
    const size_t smem = static_cast<size_t>(per) * 16;
    if (a.dtype == GTO_BF16) e = launch_stream<Bf16>(a, C, smem, stream);
    else if (a.dtype == GTO_F16) e = launch_stream<F16>(a, C, smem, stream);
    else e = launch_stream<F32>(a, C, smem, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    if (a.d2t == nullptr) return cudaGetLastError();
  }
  // any injective map (the streaming kernel has returned at once if the map is increasing,
  // this one returns at once if it is), and rows too long for a cluster's shared memory
  TokenLossArgs g = a;
  if (C == 0) g.map_state = nullptr;
  if (a.dtype == GTO_BF16)
    token_loss_gather_kernel<Bf16><<<a.B, kTokThreads, 0, stream>>>(g);
  else if (a.dtype == GTO_F16)
    token_loss_gather_kernel<F16><<<a.B, kTokThreads, 0, stream>>>(g);
  else
    token_loss_gather_kernel<F32><<<a.B, kTokThreads, 0, stream>>>(g);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
