// Row pass: log-sum-exp and exact top-k (value descending, id ascending) of V-wide logit
// rows.  Serves the draft rows (Sec. 3.1 (i): the k best tokens of every expansion) and,
// with k = 1, the target rows (log-sum-exp for the probabilities of Eq. 4 and the greedy
// target token).  One CTA per row; every logit byte is read once from HBM.
//
// Log-sum-exp: a thread sums 2^(z*log2e - ref).  The reference starts as log2e times the
// largest of the first logits its warp loads (a sample of ~1000, so it sits close to the row
// maximum and all threads of a warp normally share it); a thread whose batch maximum rises
// more than kRebase (log2 units) above its reference rescales its sum and moves the
// reference up, so no argument exceeds kRebase: nothing can overflow, and the terms that
// dominate the sum have small arguments, whose fp32 rounding is small.  Thread sums are
// shifted to the warp's largest reference, the warps' sums to a common one and combined in
// fp64, and lse = ref / log2e + ln2 * log2(sum), so the fp32 rounding of log2e cancels for
// the dominant terms.
//
// Selection without sorting: while streaming, each thread keeps only the largest and the
// second largest of its batch maxima (a batch = kUnroll vectors loaded together) and which
// batch held the largest, and leaves them in shared memory at the end of the row.  One warp
// then selects: the k-th largest of the thread maxima is a lower bound tau of the row's k-th
// largest value (they are k distinct elements), so the row's top-k are among the elements
// >= tau, and only threads whose maximum reaches tau can hold any.  The best batch of such a
// thread is fetched again, a lane per 16-byte vector, so all of them share one round trip;
// if the thread's second-best batch reaches tau too, its whole share of the row is scanned
// instead.  Every element >= tau becomes a (value, id) candidate, and a candidate's rank among
// the candidates is counted directly.  A row with more candidates than the buffer holds
// (massive ties) takes k exact arg-max rounds.  Selecting on one warp instead of letting every
// warp handle its own threads costs a quarter of the instructions (the work is a dozen
// elements, but a warp pays for its divergent lanes); the log-sum-exp is finished meanwhile
// by a lane of another warp.  What the selection still costs is mostly the fetch: measured
// on B200 at 64 KB rows, the pass without any selection runs 8 % faster, of which 6 % are the
// re-fetched 32-byte sectors and the ranking, 1.6 % the hand-over and tau, 0.7 % the
// log-sum-exp epilogue.
//
// Few rows (a small batch): one CTA per row leaves most SMs idle and a CTA alone is bound
// by its own load latency, so the row is split over a thread-block cluster of kSplit CTAs,
// each running the same procedure on a slice of the vocabulary; the cluster's first CTA then
// reads the slices' partial sums and best keys through distributed shared memory and merges.
//
// The pass is bound by instruction issue as much as by HBM (one exponential per logit), so
// the streaming loop keeps the running maximum packed (two bf16 lanes per instruction) and
// warp maxima use the integer redux instruction on order-preserving keys.
#include <cooperative_groups.h>

#include "gto_common.cuh"
#include "gto_internal.h"

namespace gto {
namespace {

namespace cg = cooperative_groups;

#ifndef GTO_ROW_THREADS
#define GTO_ROW_THREADS 128
#endif
#ifndef GTO_ROW_UNROLL
#define GTO_ROW_UNROLL 4
#endif
#ifndef GTO_ROW_MIN_CTAS
#define GTO_ROW_MIN_CTAS 12  // 40 registers per thread: no spills in the streaming loop
#endif
constexpr int kThreads = GTO_ROW_THREADS;
constexpr int kWarps = kThreads / kWarp;
constexpr int kUnrollShort = GTO_ROW_UNROLL;  // vectors a thread loads together (a batch)
constexpr int kMinCtas = GTO_ROW_MIN_CTAS;    // resident CTAs per SM the register budget allows
// Long rows (the target vocabulary): six vectors per batch at 10 CTAs per SM.  Measured on
// B200 on 256 KB rows, k = 1: 7257 / 6712 GB/s (burst / sustained) against 7194 / 6646; on
// 64 KB rows the longer batches lose (6365 against 6660: five full batches and a ragged one).
#ifndef GTO_ROW_UNROLL_LONG
#define GTO_ROW_UNROLL_LONG 6
#endif
#ifndef GTO_ROW_MIN_CTAS_LONG
#define GTO_ROW_MIN_CTAS_LONG 10
#endif
constexpr int kUnrollLong = GTO_ROW_UNROLL_LONG;
constexpr int kMinCtasLong = GTO_ROW_MIN_CTAS_LONG;
constexpr int kLongRowBytes = 128 * 1024;  // rows at least this long take the long-row variant
constexpr int kCandCap = 512;  // with the rest of RowSmem: 12 CTAs stay within 132 KB per SM
constexpr float kRebase = 8.f;  // largest exponent argument before a thread moves its reference

constexpr uint32_t kKeyNegInf = 0x007fffffu;  // orderable(-inf): stands for "no element"

constexpr int kSplit = 4;  // CTAs (one cluster) per row in the split variant

// What one CTA of a split row hands to the cluster's first CTA.
struct RowPartial {
  double sum;                           // sum of 2^(z*log2e - ref) over the slice
  float ref;
  int n;                                // valid keys
  unsigned long long key[kMaxTopK];     // the slice's best (value, id) keys, descending
};

struct RowSmem {
  float tb1[kThreads];  // per thread: largest batch maximum,
  float tb2[kThreads];  //   second largest,
  int ti1[kThreads];    //   batch that held the largest
  float warp_sum[kWarps];
  float warp_ref[kWarps];
  int n_cand;
  unsigned short work[kThreads];  // threads whose best batch is fetched again
  unsigned long long cand[kCandCap];  // (value, id) keys
  unsigned long long round_best[kWarps];
  unsigned long long prev_key;
};

template <typename T>
__device__ __forceinline__ void push_candidates(RowSmem& sm, const uint4& v, int vec_index,
                                                float tau) {
  constexpr int E = T::kPerVec;
  // most vectors hold no candidate: test the vector's maximum first
  typename T::MaxAcc acc = T::max_init();
  T::max_update(acc, v);
  if (!(T::max_value(acc) >= tau)) return;
  float f[E];
  T::unpack(v, f);
#pragma unroll
  for (int e = 0; e < E; ++e) {
    if (f[e] >= tau) {
      int slot = atomicAdd(&sm.n_cand, 1);
      if (slot < kCandCap) sm.cand[slot] = make_key(f[e], vec_index * E + e);
    }
  }
}

// lse = ref / log2e + ln2 * log2(sum): log2 of the fp64 total as exponent + log2f(mantissa in
// [1,2)), so the fp32 logarithm's error stays below 1e-7.  A sum that is 0 (no terms), inf or
// NaN gives a non-finite result, which the caller reports.
__device__ __forceinline__ double lse_from_sum(float ref, double S) {
  if (S > 0.0 && S < 1e300) {
    int ex;
    const double mant = frexp(S, &ex);  // S = mant * 2^ex, mant in [0.5, 1)
    const double lg = static_cast<double>(ex - 1) +
                      static_cast<double>(log2f(static_cast<float>(mant * 2.0)));
    return static_cast<double>(ref) / static_cast<double>(kLog2e) + kLn2 * lg;
  }
  return (S == 0.0) ? -INFINITY : S;
}

// One row, or with SPLIT the slice [v_begin, v_begin + v_count) of its 16-byte vectors, by the
// whole CTA: row r of tree `tree`.  Results go to the outputs at index gid, with SPLIT to *part.
template <typename T, bool SPLIT, int kUnroll>
__device__ __forceinline__ void reduce_row(const RowReduceArgs& a, RowSmem& sm, int gid, int tree,
                                           int r, int v_begin, int v_count, RowPartial* part) {
  constexpr int E = T::kPerVec;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const char* row = static_cast<const char*>(a.logits) +
                    tensor_row(tree, r, a.R, a.pad) * a.V * T::kBytes +
                    (SPLIT ? static_cast<size_t>(v_begin) * 16 : 0);
  const int nvec = SPLIT ? v_count : a.V / E;
  const int vec0 = SPLIT ? v_begin : 0;  // vector index of the slice's first vector in the row
  const int k = a.k;

  // ---- pass 1: per-thread exponential sum; largest and second-largest batch maximum.
  //      Batches that are complete for every thread run without bounds checks.
  constexpr int kBatchVecs = kThreads * kUnroll;
  const int nfull = nvec / kBatchVecs;
  const bool ragged = nfull * kBatchVecs < nvec;
  const uint4* p = reinterpret_cast<const uint4*>(row) + tid;
  float ref = 0.f;
  float s = 0.f;
  float b1 = -INFINITY, b2 = -INFINITY;  // best and second-best batch maximum of the thread
  int i1 = 0;                            // batch that held the best
  auto load_full = [&](uint4(&v)[kUnroll], const uint4* q) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream16(q + u * kThreads);
  };
  auto load_checked = [&](uint4(&v)[kUnroll], int b) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int i = tid + b * kBatchVecs + u * kThreads;
      v[u] = make_uint4(T::kNegInfWord, T::kNegInfWord, T::kNegInfWord, T::kNegInfWord);
      if (i < nvec) v[u] = ld_stream16(reinterpret_cast<const uint4*>(row) + i);
    }
  };
  auto batch_max = [&](const uint4(&v)[kUnroll]) {
    typename T::MaxAcc acc = T::max_init();
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) T::max_update(acc, v[u]);
    return T::max_value(acc);
  };
  auto add_terms = [&](const uint4(&v)[kUnroll]) {
    // pairwise sum of a vector's terms, the vectors of the batch added together, then one add
    // into the running sum: the long chain of roundings has one link per batch, not per vector
    float batch = 0.f;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float f[E];
      T::unpack(v[u], f);
#pragma unroll
      for (int e = 0; e < E; ++e) f[e] = ex2_approx(fmaf(f[e], kLog2e, -ref));
#pragma unroll
      for (int w = 1; w < E; w <<= 1) {
#pragma unroll
        for (int e = 0; e < E; e += 2 * w) f[e] += f[e + w];
      }
      batch = u == 0 ? f[0] : batch + f[0];
    }
    s += batch;
  };
  auto track = [&](float bm, int b) {
    const float t = bm * kLog2e;
    if (t > ref + kRebase) {  // rare: keep every argument below kRebase
      s *= ex2_approx(ref - t);
      ref = t;
    }
    if (bm > b1) {  // an equal maximum counts as second best: both batches then hold candidates
      b2 = b1;
      b1 = bm;
      i1 = b;
    } else {
      b2 = fmaxf(b2, bm);
    }
  };
  {
    // first batch: its largest logit across the warp fixes the warp's reference
    uint4 v[kUnroll];
    if (nfull > 0) load_full(v, p); else load_checked(v, 0);
    b1 = batch_max(v);
    const float ref_max = from_orderable(__reduce_max_sync(kFull, orderable(b1)));
    ref = ref_max == -INFINITY ? 0.f : ref_max * kLog2e;
    add_terms(v);
  }
  for (int b = 1; b < nfull; ++b) {
    p += kBatchVecs;
    uint4 v[kUnroll];
    load_full(v, p);
    track(batch_max(v), b);
    add_terms(v);
  }
  if (ragged && nfull > 0) {
    uint4 v[kUnroll];
    load_checked(v, nfull);
    track(batch_max(v), nfull);
    add_terms(v);
  }

  // ---- hand-over: every thread's best and second-best batch maximum and best batch, and the
  //      warp's partial sum (thread sums shifted to the warp's largest reference)
  sm.tb1[tid] = b1;
  sm.tb2[tid] = b2;
  sm.ti1[tid] = i1;
  {
    const float wref = from_orderable(__reduce_max_sync(kFull, orderable(ref)));
    const float part = warp_sum_f32(s * ex2_approx(ref - wref));
    if (lane == 0) {
      sm.warp_sum[warp] = part;
      sm.warp_ref[warp] = wref;
    }
  }
  __syncthreads();

  // ---- row log-sum-exp, by the first lane of another warp while warp 0 selects: shift the
  //      warps' sums to a common reference (exact powers of two times sums that carry 2^-22
  //      already) and add them in fp64
  if (tid == (kWarps > 1 ? kWarp : 0)) {
    float Ref = -INFINITY;
    for (int w = 0; w < kWarps; ++w)
      if (sm.warp_sum[w] != 0.f) Ref = fmaxf(Ref, sm.warp_ref[w]);
    double S = 0.0;
    for (int w = 0; w < kWarps; ++w)
      if (sm.warp_sum[w] != 0.f)
        S += static_cast<double>(sm.warp_sum[w]) *
             static_cast<double>(exp2f(sm.warp_ref[w] - Ref));
    if constexpr (SPLIT) {
      part->ref = Ref;
      part->sum = S;
    } else {
      const double lse = lse_from_sum(Ref, S);
      if (!isfinite(lse)) atomicOr(a.status, kStatusNonFinite);
      a.out_lse[gid] = lse;
    }
  }

  // ---- one warp selects (the instructions of this part are paid per warp that runs it, and a
  //      row's candidates are a dozen elements): tau = the k-th largest thread maximum -- k
  //      distinct elements reach it, so the row's top-k are among the elements >= tau and only
  //      threads whose maximum reaches it can hold any.  A thread with one batch reaching tau
  //      has that batch fetched again, a lane per vector (L2 or DRAM, one round trip for all of
  //      them); with two or more its whole share of the row is scanned.
  if (warp == 0) {
    constexpr int kPerLane = kThreads / kWarp;
    const unsigned lt_mask = (1u << lane) - 1u;
    if (lane == 0) sm.n_cand = 0;
    uint32_t key[kPerLane];
#pragma unroll
    for (int q = 0; q < kPerLane; ++q) key[q] = orderable(sm.tb1[lane + 32 * q]);
    uint32_t tau_key = kKeyNegInf;
    if constexpr (kPerLane == 4) {
      // each lane sorts its four keys once; a round then takes the largest head and pops it
      // from the first lane that holds it
      auto order = [](uint32_t& x, uint32_t& y) {
        const uint32_t hi = max(x, y), lo = min(x, y);
        x = hi;
        y = lo;
      };
      order(key[0], key[1]);
      order(key[2], key[3]);
      order(key[0], key[2]);
      order(key[1], key[3]);
      order(key[1], key[2]);
      for (int round = 0; round < k; ++round) {
        tau_key = __reduce_max_sync(kFull, key[0]);
        const unsigned holders = __ballot_sync(kFull, key[0] == tau_key);
        if (lane == __ffs(holders) - 1) {
          key[0] = key[1];
          key[1] = key[2];
          key[2] = key[3];
          key[3] = 0u;  // below every key, -inf included
        }
      }
    } else {
      for (int round = 0; round < k; ++round) {  // pop the largest remaining maximum k times
        uint32_t m = key[0];
#pragma unroll
        for (int q = 1; q < kPerLane; ++q) m = max(m, key[q]);
        tau_key = __reduce_max_sync(kFull, m);
        const unsigned holders = __ballot_sync(kFull, m == tau_key);
        if (lane == __ffs(holders) - 1) {
          bool done = false;
#pragma unroll
          for (int q = 0; q < kPerLane; ++q)
            if (!done && key[q] == tau_key) {
              key[q] = 0u;  // below every key, -inf included
              done = true;
            }
        }
      }
    }
    const float tau = from_orderable(tau_key < kKeyNegInf ? kKeyNegInf : tau_key);
    int n_one = 0;
    unsigned many[kPerLane];
#pragma unroll
    for (int q = 0; q < kPerLane; ++q) {
      const int t = lane + 32 * q;
      const bool two = sm.tb2[t] >= tau;
      const bool one = sm.tb1[t] >= tau && !two;
      const unsigned m1 = __ballot_sync(kFull, one);
      if (one) sm.work[n_one + __popc(m1 & lt_mask)] = static_cast<unsigned short>(t);
      n_one += __popc(m1);
      many[q] = __ballot_sync(kFull, two);
    }
    __syncwarp();
    for (int base = 0; base < n_one * kUnroll; base += 2 * kWarp) {  // two loads in flight
      uint4 v[2];
      int idx[2];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int item = base + j * kWarp + lane;
        idx[j] = -1;
        if (item < n_one * kUnroll) {
          const int t = sm.work[item / kUnroll];
          const int i = t + sm.ti1[t] * kBatchVecs + (item % kUnroll) * kThreads;
          if (i < nvec) {
            idx[j] = i;
            v[j] = ld_stream16(row + static_cast<size_t>(i) * 16);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 2; ++j)
        if (idx[j] >= 0) push_candidates<T>(sm, v[j], vec0 + idx[j], tau);
    }
#pragma unroll
    for (int q = 0; q < kPerLane; ++q) {
      unsigned todo = many[q];
      while (todo) {
        const int t = __ffs(todo) - 1 + 32 * q;
        todo &= todo - 1;
        for (int i = t + lane * kThreads; i < nvec; i += kWarp * kThreads)
          push_candidates<T>(sm, ld_stream16(row + static_cast<size_t>(i) * 16), vec0 + i, tau);
      }
    }
  }
  __syncthreads();
  const int n_cand = sm.n_cand;

  int32_t* out_id = a.out_id + static_cast<size_t>(gid) * k;
  float* out_z = a.out_z ? a.out_z + static_cast<size_t>(gid) * k : nullptr;

  if (n_cand <= kCandCap) {
    // ---- exact top-k among the candidates: a candidate's rank is the number of larger keys
    for (int c = tid; c < n_cand; c += kThreads) {
      const uint64_t key = sm.cand[c];
      int rank = 0;
#pragma unroll 4
      for (int j = 0; j < n_cand; ++j) rank += sm.cand[j] > key ? 1 : 0;
      if (rank < k) {
        if constexpr (SPLIT) {
          part->key[rank] = key;
        } else {
          out_id[rank] = key_id(key);
          if (out_z) out_z[rank] = key_value(key);
        }
      }
    }
    if (SPLIT && tid == 0) part->n = n_cand < k ? n_cand : k;
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
          uint64_t key = make_key(f[e], (vec0 + i) * E + e);
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
        if constexpr (SPLIT) {
          part->key[round] = b;
          part->n = k;
        } else {
          out_id[round] = key_id(b);
          if (out_z) out_z[round] = key_value(b);
        }
      }
      __syncthreads();
    }
  }

}

// The first CTA of a cluster merges the slices of a split row: partial sums are shifted to
// the largest reference; the row's top-k are the best k of the slices' best keys.
template <typename T>
__device__ __forceinline__ void merge_row(const RowReduceArgs& a, cg::cluster_group& cluster,
                                          RowPartial* mine, int gid) {
  const int tid = threadIdx.x;
  const int k = a.k;
  if (tid < kSplit * kMaxTopK) {
    const RowPartial* own = cluster.map_shared_rank(mine, tid / kMaxTopK);
    const int j = tid % kMaxTopK;
    if (j < own->n) {
      const uint64_t key = own->key[j];
      int rank = 0;
      for (int c = 0; c < kSplit; ++c) {
        const RowPartial* pc = cluster.map_shared_rank(mine, c);
        const int n = pc->n;
        for (int q = 0; q < n; ++q) rank += pc->key[q] > key ? 1 : 0;
      }
      if (rank < k) {
        a.out_id[static_cast<size_t>(gid) * k + rank] = key_id(key);
        if (a.out_z) a.out_z[static_cast<size_t>(gid) * k + rank] = key_value(key);
      }
    }
  }
  if (tid == 0) {
    float Ref = -INFINITY;
    for (int c = 0; c < kSplit; ++c) {
      const RowPartial* pc = cluster.map_shared_rank(mine, c);
      if (pc->sum != 0.0) Ref = fmaxf(Ref, pc->ref);
    }
    double S = 0.0;
    for (int c = 0; c < kSplit; ++c) {
      const RowPartial* pc = cluster.map_shared_rank(mine, c);
      if (pc->sum != 0.0) S += pc->sum * static_cast<double>(exp2f(pc->ref - Ref));
    }
    const double lse = lse_from_sum(Ref, S);
    if (!isfinite(lse)) atomicOr(a.status, kStatusNonFinite);
    a.out_lse[gid] = lse;
  }
}

// Rows come either as (row in tree, tree) = (blockIdx.x, blockIdx.y), one per CTA, or from
// the work list, which a bounded 1-D grid walks with a stride: the list's length is known
// on the device only, and a CTA per possible entry would launch ~100 000 CTAs that exit at
// once (measured: 0.54 ns each, 53 us per launch at the paper's shapes).
template <typename T, int U, int CTAS>
__global__ void __launch_bounds__(kThreads, CTAS) row_reduce_kernel(RowReduceArgs a) {
  __shared__ RowSmem sm;
  if (a.list == nullptr) {
    reduce_row<T, false, U>(a, sm, blockIdx.y * a.R + blockIdx.x, blockIdx.y, blockIdx.x, 0, 0, nullptr);
    return;
  }
  const int count = *a.list_count;
  for (int li = blockIdx.x; li < count; li += gridDim.x) {
    const int gid = a.list[li];
    const int tree = a.pad != 0 ? gid / a.R : 0;  // a tensor without padding rows needs no split
    reduce_row<T, false, U>(a, sm, gid, tree, gid - tree * a.R, 0, 0, nullptr);
    __syncthreads();  // the row's shared state is read to the end before the next row starts
  }
}

// The same with every row split over a cluster of kSplit CTAs (grid.x counts CTAs: kSplit per
// row or per list walker).
template <typename T>
__global__ void __cluster_dims__(kSplit, 1, 1) __launch_bounds__(kThreads, kMinCtas)
    row_reduce_split_kernel(RowReduceArgs a) {
  __shared__ RowSmem sm;
  __shared__ RowPartial part;
  cg::cluster_group cluster = cg::this_cluster();
  const int slice = static_cast<int>(cluster.block_rank());
  const int nvec = a.V / T::kPerVec;
  const int per_slice = (nvec + kSplit - 1) / kSplit;
  const int v_begin = min(slice * per_slice, nvec);
  const int v_count = min(per_slice, nvec - v_begin);
  const int walker = blockIdx.x / kSplit, walkers = gridDim.x / kSplit;
  const int count = a.list != nullptr ? *a.list_count : 1;
  for (int li = a.list != nullptr ? walker : 0; li < count; li += walkers) {
    int gid, tree, r;
    if (a.list != nullptr) {
      gid = a.list[li];
      tree = a.pad != 0 ? gid / a.R : 0;
      r = gid - tree * a.R;
    } else {
      r = walker;
      tree = blockIdx.y;
      gid = tree * a.R + r;
    }
    reduce_row<T, true, kUnrollShort>(a, sm, gid, tree, r, v_begin, v_count, &part);
    cluster.sync();  // every slice's partial is complete and visible
    if (slice == 0) merge_row<T>(a, cluster, &part, gid);
    cluster.sync();  // nobody rewrites or leaves before the merge has read the partials
  }
}

}  // namespace

cudaError_t launch_row_reduce(const RowReduceArgs& a, cudaStream_t stream, int64_t* launches) {
  if (a.n_rows <= 0) return cudaSuccess;
  dim3 grid(a.n_rows), block(kThreads);
  if (a.list != nullptr && a.grid_cap > 0 && a.n_rows > a.grid_cap) grid = dim3(a.grid_cap);
  if (a.list == nullptr) {
    if (a.n_rows % a.R != 0 || a.n_rows / a.R > 65535) return cudaErrorInvalidValue;
    grid = dim3(a.R, a.n_rows / a.R);
  }
  if (a.n_rows <= a.split_below) {
    // a small batch: kSplit CTAs per row
    grid.x *= kSplit;
    if (a.dtype == GTO_BF16)
      row_reduce_split_kernel<Bf16><<<grid, block, 0, stream>>>(a);
    else if (a.dtype == GTO_F16)
      row_reduce_split_kernel<F16><<<grid, block, 0, stream>>>(a);
    else
      row_reduce_split_kernel<F32><<<grid, block, 0, stream>>>(a);
  } else {
    // ... when the rows fill the device several times over (of a work list about a fifth is
    // used): with few rows the two CTAs fewer per SM cost a wave (1673 listed rows of 256 KB:
    // 89 against 82 us)
    const int64_t expected = a.list != nullptr ? a.n_rows / 5 : a.n_rows;
    const bool long_rows =
        static_cast<size_t>(a.V) * elem_bytes(a.dtype) >= static_cast<size_t>(kLongRowBytes) &&
        a.sms > 0 && expected >= 4ll * a.sms * kMinCtasLong;
    auto launch = [&](auto short_kernel, auto long_kernel) {
      if (long_rows)
        long_kernel<<<grid, block, 0, stream>>>(a);
      else
        short_kernel<<<grid, block, 0, stream>>>(a);
    };
    if (a.dtype == GTO_BF16)
      launch(row_reduce_kernel<Bf16, kUnrollShort, kMinCtas>,
             row_reduce_kernel<Bf16, kUnrollLong, kMinCtasLong>);
    else if (a.dtype == GTO_F16)
      launch(row_reduce_kernel<F16, kUnrollShort, kMinCtas>,
             row_reduce_kernel<F16, kUnrollLong, kMinCtasLong>);
    else
      launch(row_reduce_kernel<F32, kUnrollShort, kMinCtas>,
             row_reduce_kernel<F32, kUnrollLong, kMinCtasLong>);
  }
  ++*launches;
  return cudaGetLastError();
}

}  // namespace gto
