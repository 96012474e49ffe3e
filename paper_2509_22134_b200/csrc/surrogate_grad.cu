// Group-standardised advantages (Eq. 9-10), the length-normalised likelihood ratio and
// clipped surrogate (Eq. 11-12), and the gradient of the summed group losses with respect
// to the draft logits of the rows on the longest accepted sequence.
//   group_stats_kernel : one warp per group of m consecutive positions
//   grad_rows_kernel   : streams each path row once: grad = coeff * (onehot - softmax)
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kStatWarps = 4;

__device__ __forceinline__ double wsum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

__global__ void __launch_bounds__(kStatWarps * 32) group_stats_kernel(GradArgs a) {
  const int lane = threadIdx.x & 31;
  const int grp = blockIdx.x * kStatWarps + (threadIdx.x >> 5);
  const int m = a.m, B = a.B, D = a.D;
  if (grp >= B / m) return;
  const int b0 = grp * m;
  const bool debias = !(a.flags & GTO_FLAG_NO_DEBIAS);
  // Eq. 9
  double sum = 0.0;
  for (int i = lane; i < m; i += 32) {
    int b = b0 + i;
    double R = a.reward.reward[b] - (debias ? a.reward.reward[B + b] : 0.0);
    a.out.R[b] = R;
    sum += R;
  }
  const double mean = wsum(sum) / m;
  double sq = 0.0;
  for (int i = lane; i < m; i += 32) {
    int b = b0 + i;
    double R = a.reward.reward[b] - (debias ? a.reward.reward[B + b] : 0.0);
    sq += (R - mean) * (R - mean);
  }
  const bool unbiased = (a.flags & GTO_FLAG_STD_UNBIASED) && m > 1;
  const double sd = sqrt(wsum(sq) / (unbiased ? m - 1 : m));
  const double eps = static_cast<double>(a.clip_eps);
  double loss = 0.0;
  for (int i = lane; i < m; i += 32) {
    int b = b0 + i;
    double R = a.reward.reward[b] - (debias ? a.reward.reward[B + b] : 0.0);
    double A = (R - mean) / (sd + static_cast<double>(a.std_delta));  // Eq. 10
    int l = a.reward.path_len[b];
    if (l < 0 || l > D) {  // a path has at most D steps
      atomicOr(a.status, kStatusBadIndex);
      l = 0;
    }
    double diff = 0.0, cur = 0.0, old = 0.0;
    for (int j = 0; j < l; ++j) {
      cur += static_cast<double>(a.reward.path_logp[b * D + j]);
      old += static_cast<double>(a.old_logp[b * D + j]);
    }
    diff = cur - old;
    int lden = l > 1 ? l : 1;
    double s = exp(diff / lden);  // Eq. 11
    double clipped = fmin(fmax(s, 1.0 - eps), 1.0 + eps);
    loss += -(1.0 / m) * fmin(s * A, clipped * A);  // Eq. 12
    bool active = (A >= 0.0 && s <= 1.0 + eps) || (A < 0.0 && s >= 1.0 - eps);
    a.out.adv[b] = A;
    a.out.ratio[b] = s;
    a.out.active[b] = active ? 1 : 0;
    const double coeff =
        active ? static_cast<double>(a.grad_scale) * (-1.0 / m) * A * s / lden : 0.0;
    a.out.coeff[b] = coeff;
    // the rows that carry a gradient, for the list-walking gradient kernel (the same test
    // as there: the coefficient as fp32)
    if (a.live_list != nullptr && static_cast<float>(coeff) != 0.f && l > 0) {
      const int at = atomicAdd(a.live_count, l);
      for (int j = 0; j < l; ++j) a.live_list[at + j] = b * D + j;
    }
  }
  loss = wsum(loss);
  if (lane == 0) a.out.loss[grp] = loss;
}

constexpr int kGradThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kGradThreads) grad_rows_kernel(GradArgs a) {
  constexpr int E = T::kPerVec;
  const int bj = blockIdx.x;
  const int b = bj / a.D, j = bj - b * a.D;
  const int nvec = a.V / E;
  const int per = (nvec + gridDim.y - 1) / gridDim.y;
  const int v0 = blockIdx.y * per;
  const int v1 = min(nvec, v0 + per);
  char* out = static_cast<char*>(a.grad) + static_cast<size_t>(bj) * a.V * T::kBytes;
  const int l = a.reward.path_len[b];
  const float c = static_cast<float>(a.out.coeff[b]);
  if (j >= l || c == 0.f) {
    if (a.flags & GTO_FLAG_GRAD_LIVE_ROWS) return;  // the caller reads live rows only
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int i = v0 + threadIdx.x; i < v1; i += kGradThreads)
      st_stream16(out + static_cast<size_t>(i) * 16, zero);
    return;
  }
  const int row = a.reward.path_row[bj];
  const int tok = a.reward.path_token[bj];
  if (row < 0 || row >= a.R) {  // not a context row: report, write nothing from it
    if (threadIdx.x == 0) atomicOr(a.status, kStatusBadIndex);
    return;
  }
  const float nref =
      -static_cast<float>(a.row_lse[static_cast<size_t>(b) * a.R + row] * 1.4426950408889634);
  const char* in = static_cast<const char*>(a.draft) +
                   tensor_row(b, row, a.R, a.k - 1) * a.V * T::kBytes;
  for (int i = v0 + threadIdx.x; i < v1; i += kGradThreads) {
    uint4 v = ld_stream16(in + static_cast<size_t>(i) * 16);
    float f[E];
    T::unpack(v, f);
#pragma unroll
    for (int e = 0; e < E; ++e) {
      float sm = ex2_approx(fmaf(f[e], kLog2e, nref));
      f[e] = -c * sm;
    }
    int rel = tok - i * E;
    if (rel >= 0 && rel < E) {
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (e == rel) f[e] += c;
    }
    st_stream16(out + static_cast<size_t>(i) * 16, T::pack(f));
  }
}

// The same rows from the list group_stats_kernel made: a bounded grid walks (row, quarter of
// the row) units, so no CTA is launched for the ~93 % of the slices that carry no gradient.
constexpr int kLiveParts = 4;

template <typename T>
__global__ void __launch_bounds__(kGradThreads) grad_live_rows_kernel(GradArgs a) {
  constexpr int E = T::kPerVec;
  constexpr int U = 4;  // vectors in flight per thread
  const int nvec = a.V / E;
  const int per = (nvec + kLiveParts - 1) / kLiveParts;
  const int units = *a.live_count * kLiveParts;
  for (int unit = blockIdx.x; unit < units; unit += gridDim.x) {
    const int bj = a.live_list[unit / kLiveParts];
    const int part = unit % kLiveParts;
    const int b = bj / a.D;
    const int row = a.reward.path_row[bj];
    const int tok = a.reward.path_token[bj];
    if (row < 0 || row >= a.R) {  // not a context row: report, write nothing from it
      if (threadIdx.x == 0) atomicOr(a.status, kStatusBadIndex);
      continue;
    }
    const float c = static_cast<float>(a.out.coeff[b]);
    const float nref =
        -static_cast<float>(a.row_lse[static_cast<size_t>(b) * a.R + row] * 1.4426950408889634);
    const char* in = static_cast<const char*>(a.draft) +
                     tensor_row(b, row, a.R, a.k - 1) * a.V * T::kBytes;
    char* out = static_cast<char*>(a.grad) + static_cast<size_t>(bj) * a.V * T::kBytes;
    const int v1 = min(nvec, (part + 1) * per);
    for (int i0 = part * per + threadIdx.x; i0 < v1; i0 += U * kGradThreads) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * kGradThreads;
        if (i < v1) v[u] = ld_stream16(in + static_cast<size_t>(i) * 16);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * kGradThreads;
        if (i >= v1) break;
        float f[E];
        T::unpack(v[u], f);
#pragma unroll
        for (int e = 0; e < E; ++e) f[e] = -c * ex2_approx(fmaf(f[e], kLog2e, nref));
        const int rel = tok - i * E;
        if (rel >= 0 && rel < E) {
#pragma unroll
          for (int e = 0; e < E; ++e)
            if (e == rel) f[e] += c;
        }
        st_stream16(out + static_cast<size_t>(i) * 16, T::pack(f));
      }
    }
  }
}

}  // namespace

cudaError_t launch_group_stats(const GradArgs& a, cudaStream_t stream, int64_t* launches) {
  int groups = a.B / a.m;
  if (a.live_list != nullptr) {
    cudaError_t e = cudaMemsetAsync(a.live_count, 0, sizeof(int32_t), stream);
    if (e != cudaSuccess) return e;
  }
  group_stats_kernel<<<(groups + kStatWarps - 1) / kStatWarps, kStatWarps * 32, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_grad_rows(const GradArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.live_list != nullptr) {
    // live rows only: a few waves of CTAs walk the list
    const dim3 grid(a.live_grid), block(kGradThreads);
    if (a.dtype == GTO_BF16)
      grad_live_rows_kernel<Bf16><<<grid, block, 0, stream>>>(a);
    else if (a.dtype == GTO_F16)
      grad_live_rows_kernel<F16><<<grid, block, 0, stream>>>(a);
    else
      grad_live_rows_kernel<F32><<<grid, block, 0, stream>>>(a);
    ++*launches;
    return cudaGetLastError();
  }
  int vec_per_row = a.V / (16 / elem_bytes(a.dtype));
  int split = (vec_per_row + kGradThreads * 8 - 1) / (kGradThreads * 8);  // ~8 vectors/thread
  if (split < 1) split = 1;
  if (split > 64) split = 64;
  dim3 grid(a.B * a.D, split), block(kGradThreads);
  if (a.dtype == GTO_BF16)
    grad_rows_kernel<Bf16><<<grid, block, 0, stream>>>(a);
  else if (a.dtype == GTO_F16)
    grad_rows_kernel<F16><<<grid, block, 0, stream>>>(a);
  else
    grad_rows_kernel<F32><<<grid, block, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
