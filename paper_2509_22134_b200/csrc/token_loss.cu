// Token-level loss of Eq. 13 / App. B: for every position the cross-entropy
// H(p_T, p_M) = -sum_v p_T(v) log p_M(v) between the target's and the draft's next-token
// distributions under the same teacher-forced prefix (the root context row of the current
// draft's tree), and its derivative weight * (p_M - p_T) with respect to the draft logits.
// With a reduced draft vocabulary the target distribution is the softmax of the target
// logits at the mapped ids.
//
// Streaming kernel (token_loss_stream_kernel): a position is shared by a thread-block
// cluster; every CTA owns a contiguous range of draft ids.  Pass A brings the range's target
// logits into shared memory in draft-id order -- without an id map with 16-byte streaming
// loads; with one by a gather through L1 in which one warp load covers 32 neighbouring draft
// ids, whose target ids lie within a few 128-byte lines, so that every 32-byte sector of the
// target row comes from HBM once (a vocabulary subset listed in id order touches all of them:
// the bytes moved are those of the whole row) -- and sums their exponentials from shared
// memory; the cluster then combines the partial sums through distributed shared memory.
// Pass B streams the draft row once, takes the target logits from shared memory, and writes
// the gradient row.  Any map is served; an id outside the target vocabulary is reported in
// the status word and counts as probability 0.
//
// Two-pass kernel (token_loss_gather_kernel): one CTA per position, two passes over the two
// rows (the second hits L2), nothing kept in shared memory.  Serves short rows without a map
// in a large batch, where it is faster, and rows too long for a cluster's shared memory.
#include <cooperative_groups.h>

#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

namespace cg = cooperative_groups;

#ifndef GTO_TOK_THREADS
#define GTO_TOK_THREADS 256
#endif
constexpr int kTokThreads = GTO_TOK_THREADS;  // two-pass kernel
constexpr int kTokWarps = kTokThreads / 32;
#ifndef GTO_TOK_STREAM_THREADS
#define GTO_TOK_STREAM_THREADS 512
#endif
constexpr int kStreamMaxThreads = 512;  // streaming kernel: the block size is a launch parameter
constexpr int kStreamMaxWarps = kStreamMaxThreads / 32;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// ------------------------------------------------------------------ streaming kernel
struct TokPartial {
  float m;     // largest mapped target logit of the CTA's range (-inf if none)
  double s;    // sum of exp(t - m) over the range
  double h;    // the range's part of sum p_T log p_M
};

template <typename T>
__global__ void __launch_bounds__(kStreamMaxThreads, 3) token_loss_stream_kernel(TokenLossArgs a) {
  constexpr int E = T::kPerVec;
  extern __shared__ __align__(16) unsigned char s_raw[];  // the range's target logits, logit dtype
  __shared__ TokPartial part;
  __shared__ float s_m[kStreamMaxWarps];
  __shared__ double s_s[kStreamMaxWarps];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = static_cast<int>(cluster.num_blocks());
  const int c = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_threads = blockDim.x, n_warps = n_threads >> 5;

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
    for (int i = vec0 + tid; i < vec1; i += n_threads) {
      reinterpret_cast<uint4*>(s_raw)[i - vec0] = ld_stream16(zt + static_cast<size_t>(i) * 16);
    }
  } else if (id1 > id0) {
    // gather through L1: lane l of a warp takes draft ids base + e*32 + l, so that one warp load
    // covers 32 neighbouring draft ids, whose target ids lie within a few 128-byte lines
    // (a sector is fetched from L2 once and hit again by the following loads)
    constexpr int kChunk = 32 * E;
#ifndef GTO_TOK_UC
#define GTO_TOK_UC 2
#endif
    constexpr int UC = GTO_TOK_UC;  // chunks in flight per warp
    const int n_ids = id1 - id0;
    const Elem* zt_e = reinterpret_cast<const Elem*>(zt);
    for (int c0 = warp * UC * kChunk; c0 < n_ids; c0 += n_warps * UC * kChunk) {
      int id[UC][E];
#pragma unroll
      for (int u = 0; u < UC; ++u)
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const int v = c0 + u * kChunk + e * 32 + lane;
          id[u][e] = v < n_ids ? __ldg(a.d2t + id0 + v) : -1;
        }
      Elem x[UC][E];
      bool bad = false;
#pragma unroll
      for (int u = 0; u < UC; ++u)
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const int v = c0 + u * kChunk + e * 32 + lane;
          x[u][e] = T::kNegInfElem;  // an id outside the target vocabulary: probability 0
          if (static_cast<unsigned>(id[u][e]) < static_cast<unsigned>(a.V_target))
            x[u][e] = zt_e[id[u][e]];
          else if (v < n_ids)
            bad = true;
        }
#pragma unroll
      for (int u = 0; u < UC; ++u)
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const int v = c0 + u * kChunk + e * 32 + lane;
          if (v < n_ids) s_t[v] = x[u][e];
        }
      if (bad) atomicOr(a.status, kStatusBadIndex);
    }
  }
  __syncthreads();
  // the range's log-sum-exp from shared memory (dense, in draft-id order)
  for (int i = tid; i < vec1 - vec0; i += n_threads) {
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
    for (int w = 1; w < n_warps; ++w) M = fmaxf(M, s_m[w]);
    double S = 0.0;
    for (int w = 0; w < n_warps; ++w)
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
  for (int i = vec0 + tid; i < vec1; i += n_threads) {
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
    for (int w = 0; w < n_warps; ++w) H += s_s[w];
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
cudaError_t launch_stream(const TokenLossArgs& a, int C, int threads, size_t smem,
                          cudaStream_t stream) {
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
  cfg.blockDim = dim3(threads);
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
  if (C > 0) {
    const int E = 16 / elem_bytes(a.dtype);
    const int per = (a.V_draft / E + C - 1) / C;
    const size_t smem = static_cast<size_t>(per) * 16;
    // measured on B200 (us per call, bf16): B = 1024 with a map 512 threads 99, 256 threads
    // 117; without a map (151 936 ids) 512 threads 152, 256 threads 162; B = 64 with a map
    // 512 threads 27, 256 threads 16
    const int threads = a.B >= 2 * sms ? GTO_TOK_STREAM_THREADS : 256;
    if (a.dtype == GTO_BF16) e = launch_stream<Bf16>(a, C, threads, smem, stream);
    else if (a.dtype == GTO_F16) e = launch_stream<F16>(a, C, threads, smem, stream);
    else e = launch_stream<F32>(a, C, threads, smem, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    return cudaGetLastError();
  }
  // short unmapped rows of a large batch, and rows too long for a cluster's shared memory
  if (a.dtype == GTO_BF16)
    token_loss_gather_kernel<Bf16><<<a.B, kTokThreads, 0, stream>>>(a);
  else if (a.dtype == GTO_F16)
    token_loss_gather_kernel<F16><<<a.B, kTokThreads, 0, stream>>>(a);
  else
    token_loss_gather_kernel<F32><<<a.B, kTokThreads, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
