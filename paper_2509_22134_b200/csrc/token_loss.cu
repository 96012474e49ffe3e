// Token-level loss of Eq. 13 / App. B: for every position the cross-entropy
// H(p_T, p_M) = -sum_v p_T(v) log p_M(v) between the target's and the draft's next-token
// distributions under the same teacher-forced prefix (the root context row of the current
// draft's tree), and its derivative weight * (p_M - p_T) with respect to the draft logits.
// With a reduced draft vocabulary the target distribution is the softmax of the target
// logits at the mapped ids.  One CTA per position, two passes over the two rows (the second
// hits L2): log-sum-exp of the mapped target logits, then loss and gradient.  The id-map
// gather is laid out so that a warp load touches few 32-byte sectors (the gather is bound by
// L1 wavefronts otherwise: 31 sectors per request were measured with ids dealt 8 per lane).
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kTokThreads = 256;
constexpr int kTokWarps = kTokThreads / 32;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

template <typename T>
__global__ void __launch_bounds__(kTokThreads, 8) token_loss_kernel(TokenLossArgs a) {
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
  char* out = static_cast<char*>(a.grad_root) + static_cast<size_t>(b) * a.V_draft * T::kBytes;
  float h = 0.f;
  for (int c = warp; c < nchunk; c += kTokWarps) {
    float t[E], z[E];
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
#pragma unroll
      for (int e = 0; e < E; ++e) {
        const float lq = z[e] - lse_d;                               // log p_M
        const float pt = ex2_approx((t[e] - lse_t) * kLog2e);       // p_T
        h = fmaf(pt, lq, h);
        z[e] = a.weight * (ex2_approx(lq * kLog2e) - pt);
      }
      st_stream16(out + static_cast<size_t>(i) * 16, T::pack(z));
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

}  // namespace

cudaError_t launch_token_loss(const TokenLossArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.B <= 0) return cudaSuccess;
  if (a.dtype == GTO_BF16)
    token_loss_kernel<Bf16><<<a.B, kTokThreads, 0, stream>>>(a);
  else if (a.dtype == GTO_F16)
    token_loss_kernel<F16><<<a.B, kTokThreads, 0, stream>>>(a);
  else
    token_loss_kernel<F32><<<a.B, kTokThreads, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
