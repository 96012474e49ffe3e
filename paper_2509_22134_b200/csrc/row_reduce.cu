// Row pass: log-sum-exp and exact top-k (value descending, id ascending) of V-wide logit
// rows.  Serves the draft rows (Sec. 3.1 (i): the k best tokens of every expansion) and,
// with k = 1, the target rows (log-sum-exp for the probabilities of Eq. 4 and the greedy
// target token).  One CTA per row; every logit byte is read once from HBM.
//
// Selection without sorting: while streaming, each thread keeps only the running maximum
// of its own elements.  The k-th largest of the thread maxima is a lower bound tau of the
// row's k-th largest value (those maxima are k distinct elements), so the row's top-k are
// among the elements >= tau, and only threads whose maximum reaches tau can hold any.
// Those few threads rescan their own vectors (L2 hits) and push (value, id) candidates;
// one warp then extracts the k best keys exactly.  A row with more candidates than the
// buffer holds (massive ties) takes k exact arg-max rounds over the row instead.
#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;
constexpr int kUnroll = 4;
constexpr int kCandCap = 1024;

struct RowSmem {
  float warp_top[kWarps][kMaxTopK];  // each warp's k largest thread maxima, descending
  float warp_ref[kWarps];            // log2-domain reference of the warp's partial sum
  float warp_sum[kWarps];
  float tau;
  int n_cand;
  float cand_z[kCandCap];
  int cand_id[kCandCap];
  unsigned long long round_best[kWarps];
  unsigned long long prev_key;
};

// Descending bitonic sort of one value per lane.
__device__ __forceinline__ float warp_sort_desc(float v, int lane) {
#pragma unroll
  for (int k2 = 2; k2 <= 32; k2 <<= 1) {
#pragma unroll
    for (int j = k2 >> 1; j > 0; j >>= 1) {
      float o = __shfl_xor_sync(kFull, v, j);
      bool desc = (lane & k2) == 0;
      bool lower = (lane & j) == 0;
      v = (lower == desc) ? fmaxf(v, o) : fminf(v, o);
    }
  }
  return v;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) row_reduce_kernel(RowReduceArgs a) {
  constexpr int E = T::kPerVec;
  __shared__ RowSmem sm;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;

  int gid = blockIdx.x;
  if (a.list != nullptr) {
    if (gid >= *a.list_count) return;
    gid = a.list[gid];
  }
  const int tree = gid / a.R;
  const int r = gid - tree * a.R;
  const char* row =
      static_cast<const char*>(a.logits) + tensor_row(tree, r, a.R, a.pad) * a.V * T::kBytes;
  const int nvec = a.V / E;
  const int k = a.k;

  // ---- pass 1: per-thread running maximum and sum of 2^(z*log2e - ref)
  float m = -INFINITY, ref = -INFINITY, s = 0.f;
  for (int i0 = tid; i0 < nvec; i0 += kThreads * kUnroll) {
    uint4 v[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int i = i0 + u * kThreads;
      v[u] = (i < nvec) ? ld_stream16(row + static_cast<size_t>(i) * 16)
                        : make_uint4(T::kNegInfWord, T::kNegInfWord, T::kNegInfWord,
                                     T::kNegInfWord);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float f[E];
      T::unpack(v[u], f);
      float vmax = f[0];
#pragma unroll
      for (int e = 1; e < E; ++e) vmax = fmaxf(vmax, f[e]);
      if (vmax > m) {
        float nref = vmax * kLog2e;
        s *= ex2_approx(ref - nref);
        m = vmax;
        ref = nref;
      }
#pragma unroll
      for (int e = 0; e < E; ++e) s += ex2_approx(fmaf(f[e], kLog2e, -ref));
    }
  }

  // ---- warp level: k largest thread maxima, and the warp's partial sum
  {
    float sorted = warp_sort_desc(m, lane);
    if (lane < k) sm.warp_top[warp][lane] = sorted;
    float wref = warp_max_f32(ref);
    float part = (ref == -INFINITY) ? 0.f : s * ex2_approx(ref - wref);
    part = warp_sum_f32(part);
    if (lane == 0) {
      sm.warp_ref[warp] = wref;
      sm.warp_sum[warp] = part;
    }
  }
  if (tid == 0) sm.n_cand = 0;
  __syncthreads();

  // ---- warp 0: tau = k-th largest thread maximum (with multiplicity)
  if (warp == 0) {
    constexpr int kPer = (kWarps * kMaxTopK + 31) / 32;
    float mine[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      int idx = lane + q * 32;
      int w = idx / kMaxTopK, c = idx % kMaxTopK;
      mine[q] = (w < kWarps && c < k) ? sm.warp_top[w][c] : -INFINITY;
    }
    float tau = -INFINITY;
    for (int round = 0; round < k; ++round) {
      float best = mine[0];
#pragma unroll
      for (int q = 1; q < kPer; ++q) best = fmaxf(best, mine[q]);
      float wbest = warp_max_f32(best);
      tau = wbest;
      unsigned holders = __ballot_sync(kFull, best == wbest);
      if (lane == __ffs(holders) - 1) {  // drop one instance
        bool done = false;
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
          if (!done && mine[q] == wbest) {
            mine[q] = -INFINITY;
            done = true;
          }
        }
      }
    }
    if (lane == 0) sm.tau = tau;
  }
  __syncthreads();
  const float tau = sm.tau;

  // ---- pass 2: threads that can hold a top-k element rescan their own vectors
  if (m >= tau) {
    for (int i = tid; i < nvec; i += kThreads) {
      uint4 v = ld_stream16(row + static_cast<size_t>(i) * 16);
      float f[E];
      T::unpack(v, f);
#pragma unroll
      for (int e = 0; e < E; ++e) {
        if (f[e] >= tau) {
          int slot = atomicAdd(&sm.n_cand, 1);
          if (slot < kCandCap) {
            sm.cand_z[slot] = f[e];
            sm.cand_id[slot] = i * E + e;
          }
        }
      }
    }
  }
  __syncthreads();
  const int n_cand = sm.n_cand;

  int32_t* out_id = a.out_id + static_cast<size_t>(gid) * k;
  float* out_z = a.out_z ? a.out_z + static_cast<size_t>(gid) * k : nullptr;

  if (n_cand <= kCandCap) {
    // ---- exact top-k among the candidates: k rounds of warp arg-max on (value, id) keys
    if (warp == 0) {
      uint64_t prev = ~0ull;
      for (int round = 0; round < k; ++round) {
        uint64_t best = 0;
        for (int c = lane; c < n_cand; c += 32) {
          uint64_t key = make_key(sm.cand_z[c], sm.cand_id[c]);
          if (key < prev && key > best) best = key;
        }
        best = warp_max_u64(best);
        prev = best;
        if (lane == 0) {
          out_id[round] = key_id(best);
          if (out_z) out_z[round] = key_value(best);
        }
      }
    }
  } else {
    // ---- too many ties at tau: k exact arg-max rounds over the whole row
    if (tid == 0) sm.prev_key = ~0ull;
    __syncthreads();
    for (int round = 0; round < k; ++round) {
      const uint64_t prev = sm.prev_key;
      uint64_t best = 0;
      for (int i = tid; i < nvec; i += kThreads) {
        uint4 v = ld_stream16(row + static_cast<size_t>(i) * 16);
        float f[E];
        T::unpack(v, f);
#pragma unroll
        for (int e = 0; e < E; ++e) {
          uint64_t key = make_key(f[e], i * E + e);
          if (key < prev && key > best) best = key;
        }
      }
      best = warp_max_u64(best);
      if (lane == 0) sm.round_best[warp] = best;
      __syncthreads();
      if (tid == 0) {
        uint64_t b = 0;
        for (int w = 0; w < kWarps; ++w) b = sm.round_best[w] > b ? sm.round_best[w] : b;
        sm.prev_key = b;
        out_id[round] = key_id(b);
        if (out_z) out_z[round] = key_value(b);
      }
      __syncthreads();
    }
  }

  // ---- row log-sum-exp: combine the warps in fp64
  if (tid == 0) {
    float Ref = sm.warp_ref[0];
    for (int w = 1; w < kWarps; ++w) Ref = fmaxf(Ref, sm.warp_ref[w]);
    double S = 0.0;
    for (int w = 0; w < kWarps; ++w) {
      if (sm.warp_ref[w] != -INFINITY)
        S += static_cast<double>(sm.warp_sum[w]) *
             exp2(static_cast<double>(sm.warp_ref[w]) - static_cast<double>(Ref));
    }
    double lse = (static_cast<double>(Ref) + log2(S)) * kLn2;
    if (!isfinite(lse)) atomicOr(a.status, kStatusNonFinite);
    a.out_lse[gid] = lse;
  }
}

}  // namespace

cudaError_t launch_row_reduce(const RowReduceArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.n_rows <= 0) return cudaSuccess;
  dim3 grid(a.n_rows), block(kThreads);
  if (a.dtype == GTO_BF16)
    row_reduce_kernel<Bf16><<<grid, block, 0, stream>>>(a);
  else
    row_reduce_kernel<F32><<<grid, block, 0, stream>>>(a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
