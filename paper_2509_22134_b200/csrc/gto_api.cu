// C ABI of the GTO draft-tree pass: argument validation, workspace, launch sequencing.
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gto_common.cuh"
#include "gto_internal.h"

struct gto_ctx {
  gto_config cfg;
  int device;
  int R, P;
  int row_grid_cap;   // CTAs for the listed-row pass: a few waves of the device
  int row_split_rows;   // batches with at most this many rows may split every row over a cluster
  char* ws;           // one allocation
  int32_t* top_id;    // [G*B*R, k] draft row top-k ids
  float* top_z;       // [G*B*R, k] draft row top-k logits
  int32_t* list;      // [G*B*R] needed target rows
  int32_t* list_count;
  int32_t* status;
  int32_t* live_list;   // gradient: slices that carry a gradient (GTO_FLAG_GRAD_LIVE_ROWS)
  int32_t* live_count;
  int sms;
  int32_t* h_list;    // page-locked host copy of the work list: [0] = count, then the rows
  int64_t last_host_rows;
  int64_t launches;
  bool timing;
  struct Span { cudaEvent_t t0, t1; int kernel; };
  std::vector<Span> spans;   // event pairs, reused across reads
  size_t spans_used;
};

#ifndef GTO_ROW_SPLIT_ROWS_PER_SM
#define GTO_ROW_SPLIT_ROWS_PER_SM 10  // up to this many rows per SM, a row is split over a cluster
#endif
#ifndef GTO_ROW_GRID_WAVES
#define GTO_ROW_GRID_WAVES 16  // resident-CTA waves launched for the listed-row pass (measured best of 1..24)
#endif

namespace {

size_t align_up(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

// Brackets one kernel launch with two events when per-kernel timing is on.
struct LaunchSpan {
  gto_ctx* c;
  cudaStream_t s;
  long index = -1;  // into c->spans (an index survives the vector growing)
  LaunchSpan(gto_ctx* ctx, int kernel, cudaStream_t stream) : c(ctx), s(stream) {
    if (!c->timing) return;
    if (c->spans_used == c->spans.size()) {
      gto_ctx::Span n{};
      if (cudaEventCreate(&n.t0) != cudaSuccess) return;
      if (cudaEventCreate(&n.t1) != cudaSuccess) {
        cudaEventDestroy(n.t0);
        return;
      }
      c->spans.push_back(n);
    }
    index = static_cast<long>(c->spans_used++);
    c->spans[index].kernel = kernel;
    cudaEventRecord(c->spans[index].t0, s);
  }
  ~LaunchSpan() {
    if (index >= 0) cudaEventRecord(c->spans[index].t1, s);
  }
};

// NVTX range around one library call (a no-op unless a profiler is attached).
struct CallRange {
  explicit CallRange(const char* name) { nvtxRangePushA(name); }
  ~CallRange() { nvtxRangePop(); }
};

// Rows are split over a cluster only where that was measured to pay: few rows (at most
// GTO_ROW_SPLIT_ROWS_PER_SM per SM) that are long (slices of at least 32 KB).  At the paper's
// shapes that is the target pass below 8 positions and 300 KB draft rows of small batches; 64 KB
// draft rows are faster unsplit at any batch size (22 vs 46 us at 976 rows).
int split_below(const gto_ctx* ctx, int n_rows, int V) {
  const size_t row_bytes = static_cast<size_t>(V) * gto::elem_bytes(ctx->cfg.logit_dtype);
  const bool pays = n_rows <= ctx->row_split_rows && row_bytes >= 4 * 32768;
  return (pays || (ctx->cfg.flags & GTO_FLAG_FORCE_ROW_SPLIT)) ? n_rows : 0;
}

template <typename S>
bool all_set(const S* s) {
  // every member of the output structs is a pointer
  const void* const* p = reinterpret_cast<const void* const*>(s);
  for (size_t i = 0; i < sizeof(S) / sizeof(void*); ++i)
    if (p[i] == nullptr || !aligned16(p[i])) return false;
  return true;
}

}  // namespace

extern "C" {

const char* gto_status_string(gto_status s) {
  switch (s) {
    case GTO_OK: return "ok";
    case GTO_ERR_INVALID_ARG: return "invalid argument";
    case GTO_ERR_UNSUPPORTED: return "shape outside the compiled limits";
    case GTO_ERR_WORKSPACE: return "workspace allocation failed";
    case GTO_ERR_CUDA: return "CUDA runtime error";
    case GTO_ERR_NONFINITE: return "non-finite logit row";
    case GTO_ERR_TOO_LARGE: return "batch exceeds the fixed scratch of the no-allocation call";
    case GTO_ERR_BAD_INDEX: return "an index in a caller's table was out of range";
  }
  return "unknown status";
}

gto_status gto_create(gto_ctx** out, const gto_config* c, int device) {
  if (!out || !c) return GTO_ERR_INVALID_ARG;
  *out = nullptr;
  if (c->B <= 0 || c->D <= 0 || c->k <= 0 || c->g <= 0 || c->m <= 0 || c->V_draft <= 0 ||
      c->V_target <= 0)
    return GTO_ERR_INVALID_ARG;
  if (!gto::valid_dtype(c->logit_dtype)) return GTO_ERR_INVALID_ARG;
  if (c->reward_agg < GTO_AGG_LSE || c->reward_agg > GTO_AGG_MEAN) return GTO_ERR_INVALID_ARG;
  if (!(c->eta > 0.f) || !(c->clip_eps >= 0.f) || !(c->std_delta >= 0.f))
    return GTO_ERR_INVALID_ARG;
  if (c->B % c->m != 0) return GTO_ERR_INVALID_ARG;
  if (c->k > c->V_draft) return GTO_ERR_INVALID_ARG;
  const int64_t P = c->k + static_cast<int64_t>(c->D - 1) * c->k * c->k;
  if (c->g > P) return GTO_ERR_INVALID_ARG;
  if (c->G != 2) return GTO_ERR_UNSUPPORTED;
  if (c->k > gto::kMaxTopK || c->k * c->k > gto::kMaxLayer || c->g > gto::kMaxNodes ||
      c->D > gto::kMaxDepth)
    return GTO_ERR_UNSUPPORTED;
  const int eb = gto::elem_bytes(c->logit_dtype);
  if ((static_cast<int64_t>(c->V_draft) * eb) % 16 || (static_cast<int64_t>(c->V_target) * eb) % 16)
    return GTO_ERR_UNSUPPORTED;
  const int R = 1 + (c->D - 1) * c->k;
  const int64_t rows = static_cast<int64_t>(c->G) * c->B * R;
  if (rows >= (1ll << 31) / c->k) return GTO_ERR_UNSUPPORTED;
  if (static_cast<int64_t>(c->G) * c->B > 65535) return GTO_ERR_UNSUPPORTED;  // grid.y = trees

  DeviceGuard guard(device);
  if (!guard.ok) return GTO_ERR_CUDA;
  gto_ctx* ctx = new (std::nothrow) gto_ctx();
  if (!ctx) return GTO_ERR_WORKSPACE;
  ctx->cfg = *c;
  ctx->device = device;
  ctx->R = R;
  ctx->P = static_cast<int>(P);
  ctx->launches = 0;
  {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
      cudaGetLastError();
      delete ctx;
      return GTO_ERR_CUDA;
    }
    ctx->sms = sms;
    ctx->row_grid_cap = sms * 12 * GTO_ROW_GRID_WAVES;
    ctx->row_split_rows = sms * GTO_ROW_SPLIT_ROWS_PER_SM;
  }
  ctx->last_host_rows = 0;
  ctx->timing = false;
  ctx->spans_used = 0;
  size_t off = 0;
  const size_t o_id = off;  off += align_up(rows * c->k * sizeof(int32_t));
  const size_t o_z = off;   off += align_up(rows * c->k * sizeof(float));
  const size_t o_list = off; off += align_up(rows * sizeof(int32_t));
  const size_t o_live = off; off += align_up(static_cast<size_t>(c->B) * c->D * sizeof(int32_t));
  const size_t o_cnt = off; off += 256;
  const size_t o_st = off;  off += 256;
  const size_t o_lc = off;  off += 256;
  if (cudaMalloc(&ctx->ws, off) != cudaSuccess) {
    cudaGetLastError();
    delete ctx;
    return GTO_ERR_WORKSPACE;
  }
  ctx->top_id = reinterpret_cast<int32_t*>(ctx->ws + o_id);
  ctx->top_z = reinterpret_cast<float*>(ctx->ws + o_z);
  ctx->list = reinterpret_cast<int32_t*>(ctx->ws + o_list);
  ctx->list_count = reinterpret_cast<int32_t*>(ctx->ws + o_cnt);
  ctx->status = reinterpret_cast<int32_t*>(ctx->ws + o_st);
  ctx->live_list = reinterpret_cast<int32_t*>(ctx->ws + o_live);
  ctx->live_count = reinterpret_cast<int32_t*>(ctx->ws + o_lc);
  if (cudaMemset(ctx->ws + o_cnt, 0, 768) != cudaSuccess ||
      cudaMallocHost(&ctx->h_list, (rows + 1) * sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(ctx->ws);
    delete ctx;
    return GTO_ERR_WORKSPACE;
  }
  *out = ctx;
  return GTO_OK;
}

gto_status gto_destroy(gto_ctx* ctx) {
  if (!ctx) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  for (auto& sp : ctx->spans) {
    cudaEventDestroy(sp.t0);
    cudaEventDestroy(sp.t1);
  }
  cudaFreeHost(ctx->h_list);
  cudaError_t e = cudaFree(ctx->ws);
  delete ctx;
  return e == cudaSuccess ? GTO_OK : GTO_ERR_CUDA;
}

gto_status gto_build_tree(gto_ctx* ctx, const void* draft, const gto_tree* out, void* stream) {
  CallRange range("gto_build_tree");
  if (!ctx || !draft || !out || !aligned16(draft) || !all_set(out)) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  const gto_config& c = ctx->cfg;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  gto::RowReduceArgs r{};
  r.logits = draft;
  r.dtype = c.logit_dtype;
  r.V = c.V_draft;
  r.R = ctx->R;
  r.pad = c.k - 1;
  r.list = nullptr;
  r.list_count = nullptr;
  r.n_rows = c.G * c.B * ctx->R;
  r.k = c.k;
  r.out_lse = out->row_lse;
  r.out_id = ctx->top_id;
  r.out_z = ctx->top_z;
  r.status = ctx->status;
  r.split_below = split_below(ctx, r.n_rows, r.V);
  r.sms = ctx->sms;
  {
    LaunchSpan span(ctx, GTO_K_DRAFT_ROWS, s);
    if (gto::launch_row_reduce(r, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  }
  gto::TreeBuildArgs t{};
  t.n_trees = c.G * c.B;
  t.D = c.D;
  t.k = c.k;
  t.g = c.g;
  t.R = ctx->R;
  t.row_lse = out->row_lse;
  t.top_id = ctx->top_id;
  t.top_z = ctx->top_z;
  t.out = *out;
  LaunchSpan span(ctx, GTO_K_TREE_BUILD, s);
  if (gto::launch_tree_build(t, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  return GTO_OK;
}

namespace {

// Shared body of gto_tree_reward and gto_tree_reward_host.  With `target_host` the needed
// rows are first copied from there into `target` (device) at their own offsets.
gto_status tree_reward_impl(gto_ctx* ctx, const gto_tree* tree, const void* target,
                            const void* target_host, const int32_t* d2t, const gto_reward* out,
                            void* stream) {
  CallRange range(target_host ? "gto_tree_reward_host" : "gto_tree_reward");
  if (!ctx || !tree || !target || !out || !aligned16(target) || !all_set(tree) || !all_set(out))
    return GTO_ERR_INVALID_ARG;
  const gto_config& c = ctx->cfg;
  if (!d2t && c.V_draft != c.V_target) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int n_trees = c.G * c.B;
  gto::RewardPlanArgs p{};
  p.n_trees = n_trees;
  p.g = c.g;
  p.R = ctx->R;
  p.node_ctx_row = tree->node_ctx_row;
  p.list = ctx->list;
  p.list_count = ctx->list_count;
  p.row_lse_t = out->row_lse_t;
  p.row_argmax_t = out->row_argmax_t;
  p.status = ctx->status;
  {
    LaunchSpan span(ctx, GTO_K_REWARD_PLAN, s);
    if (gto::launch_reward_plan(p, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  }
  if (target_host != nullptr) {
    // the host needs the list: one synchronisation, then one copy per run of adjacent rows
    const size_t list_bytes = static_cast<size_t>(n_trees) * ctx->R * sizeof(int32_t);
    if (cudaMemcpyAsync(ctx->h_list, ctx->list_count, sizeof(int32_t), cudaMemcpyDeviceToHost, s) !=
            cudaSuccess ||
        cudaMemcpyAsync(ctx->h_list + 1, ctx->list, list_bytes, cudaMemcpyDeviceToHost, s) !=
            cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
      return GTO_ERR_CUDA;
    const int count = ctx->h_list[0];
    int32_t* rows = ctx->h_list + 1;
    std::sort(rows, rows + count);
    const size_t row_bytes = static_cast<size_t>(c.V_target) * gto::elem_bytes(c.logit_dtype);
    for (int i = 0; i < count;) {
      int j = i + 1;
      while (j < count && rows[j] == rows[j - 1] + 1) ++j;
      const size_t off = static_cast<size_t>(rows[i]) * row_bytes;
      if (cudaMemcpyAsync(static_cast<char*>(const_cast<void*>(target)) + off,
                          static_cast<const char*>(target_host) + off, (j - i) * row_bytes,
                          cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GTO_ERR_CUDA;
      i = j;
    }
    ctx->last_host_rows = count;
  }
  gto::RowReduceArgs r{};
  r.logits = target;
  r.dtype = c.logit_dtype;
  r.V = c.V_target;
  r.R = ctx->R;
  r.pad = 0;
  r.list = ctx->list;
  r.list_count = ctx->list_count;
  r.grid_cap = ctx->row_grid_cap;
  r.n_rows = n_trees * ctx->R;
  r.k = 1;
  r.out_lse = out->row_lse_t;
  r.out_id = out->row_argmax_t;
  r.out_z = nullptr;
  r.status = ctx->status;
  r.split_below = split_below(ctx, r.n_rows, r.V);
  r.sms = ctx->sms;
  {
    LaunchSpan span(ctx, GTO_K_TARGET_ROWS, s);
    if (gto::launch_row_reduce(r, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  }
  gto::RewardArgs w{};
  w.B = c.B; w.G = c.G; w.D = c.D; w.k = c.k; w.g = c.g; w.R = ctx->R;
  w.V_draft = c.V_draft;
  w.V_target = c.V_target;
  w.status = ctx->status;
  w.dtype = c.logit_dtype;
  w.agg = c.reward_agg;
  w.flags = c.flags;
  w.eta = c.eta;
  w.target = target;
  w.d2t = d2t;
  w.tree = *tree;
  w.out = *out;
  LaunchSpan span(ctx, GTO_K_TREE_REWARD, s);
  if (gto::launch_tree_reward(w, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  return GTO_OK;
}

}  // namespace

gto_status gto_tree_reward(gto_ctx* ctx, const gto_tree* tree, const void* target,
                           const int32_t* d2t, const gto_reward* out, void* stream) {
  return tree_reward_impl(ctx, tree, target, nullptr, d2t, out, stream);
}

gto_status gto_tree_reward_host(gto_ctx* ctx, const gto_tree* tree, const void* target_host,
                                void* target_dev, const int32_t* d2t, const gto_reward* out,
                                void* stream, int64_t* rows_copied) {
  if (!target_host) return GTO_ERR_INVALID_ARG;
  gto_status st = tree_reward_impl(ctx, tree, target_dev, target_host, d2t, out, stream);
  if (st == GTO_OK && rows_copied) *rows_copied = ctx->last_host_rows;
  return st;
}

gto_status gto_group_surrogate_grad(gto_ctx* ctx, const void* draft, const gto_tree* tree,
                                    const gto_reward* reward, const float* old_logp, void* grad,
                                    const gto_grad_stats* out, void* stream) {
  CallRange range("gto_group_surrogate_grad");
  if (!ctx || !draft || !tree || !reward || !old_logp || !grad || !out || !aligned16(draft) ||
      !aligned16(grad) || !aligned16(old_logp) || !all_set(tree) || !all_set(reward) ||
      !all_set(out))
    return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  const gto_config& c = ctx->cfg;
  gto::GradArgs a{};
  a.B = c.B; a.D = c.D; a.k = c.k; a.R = ctx->R; a.m = c.m; a.V = c.V_draft;
  a.dtype = c.logit_dtype;
  a.clip_eps = c.clip_eps;
  a.std_delta = c.std_delta;
  a.grad_scale = c.grad_scale;
  a.flags = c.flags;
  a.draft = draft;
  a.row_lse = tree->row_lse;
  a.reward = *reward;
  a.old_logp = old_logp;
  a.grad = grad;
  a.out = *out;
  a.status = ctx->status;
  if (c.flags & GTO_FLAG_GRAD_LIVE_ROWS) {
    a.live_list = ctx->live_list;
    a.live_count = ctx->live_count;
    a.live_grid = ctx->sms * 8;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchSpan span(ctx, GTO_K_GROUP_STATS, s);
    if (gto::launch_group_stats(a, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  }
  LaunchSpan span(ctx, GTO_K_GRAD_ROWS, s);
  if (gto::launch_grad_rows(a, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  return GTO_OK;
}

namespace {

// Shared body of gto_token_loss and gto_token_loss_accumulate.
gto_status token_loss_impl(gto_ctx* ctx, const void* draft, const void* target, const int32_t* d2t,
                           const gto_tree* tree, float weight, void* grad_out, int64_t out_stride,
                           const int32_t* acc_path_len, const double* acc_coeff,
                           const gto_token_stats* out, void* stream) {
  if (!ctx || !draft || !target || !tree || !grad_out || !out || !aligned16(draft) ||
      !aligned16(target) || !aligned16(grad_out) || !all_set(tree) || !all_set(out))
    return GTO_ERR_INVALID_ARG;
  const gto_config& c = ctx->cfg;
  if (!d2t && c.V_draft != c.V_target) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  gto::TokenLossArgs a{};
  a.B = c.B; a.k = c.k; a.R = ctx->R; a.V_draft = c.V_draft; a.V_target = c.V_target;
  a.dtype = c.logit_dtype;
  a.weight = weight;
  a.draft = draft;
  a.target = target;
  a.d2t = d2t;
  a.row_lse = tree->row_lse;
  a.grad_out = grad_out;
  a.out_stride = out_stride;
  a.acc_path_len = acc_path_len;
  a.acc_coeff = acc_coeff;
  a.loss = out->loss;
  a.lse_t = out->lse_t;
  a.status = ctx->status;
  LaunchSpan span(ctx, GTO_K_TOKEN_LOSS, s);
  if (gto::launch_token_loss(a, ctx->sms, s, &ctx->launches) != cudaSuccess) return GTO_ERR_CUDA;
  return GTO_OK;
}

}  // namespace

gto_status gto_token_loss(gto_ctx* ctx, const void* draft, const void* target, const int32_t* d2t,
                          const gto_tree* tree, float weight, void* grad_root,
                          const gto_token_stats* out, void* stream) {
  CallRange range("gto_token_loss");
  if (!ctx) return GTO_ERR_INVALID_ARG;
  return token_loss_impl(ctx, draft, target, d2t, tree, weight, grad_root, ctx->cfg.V_draft, nullptr,
                         nullptr, out, stream);
}

gto_status gto_token_loss_accumulate(gto_ctx* ctx, const void* draft, const void* target,
                                     const int32_t* d2t, const gto_tree* tree,
                                     const gto_reward* reward, const gto_grad_stats* stats,
                                     float weight, void* grad, const gto_token_stats* out,
                                     void* stream) {
  CallRange range("gto_token_loss_accumulate");
  if (!ctx || !reward || !stats || !all_set(reward) || !all_set(stats)) return GTO_ERR_INVALID_ARG;
  return token_loss_impl(ctx, draft, target, d2t, tree, weight, grad,
                         static_cast<int64_t>(ctx->cfg.D) * ctx->cfg.V_draft, reward->path_len,
                         stats->coeff, out, stream);
}

gto_status gto_sample_groups(int32_t s, int32_t m, int32_t K, const double* u, int32_t* starts) {
  if (s < 0 || m < 1 || K < 0 || static_cast<int64_t>(K) * m > s) return GTO_ERR_INVALID_ARG;
  if (K > 0 && (!u || !starts)) return GTO_ERR_INVALID_ARG;
  // choose K sorted offsets in [0, s - K m] (with repetition), then spread them by k m:
  // a bijection between such multisets and the admissible start sets
  const int64_t free_slots = static_cast<int64_t>(s) - static_cast<int64_t>(K) * m;
  for (int32_t i = 0; i < K; ++i) {
    if (!(u[i] >= 0.0 && u[i] < 1.0)) return GTO_ERR_INVALID_ARG;
    int64_t gap = static_cast<int64_t>(std::floor(u[i] * static_cast<double>(free_slots + 1)));
    starts[i] = static_cast<int32_t>(std::min(gap, free_slots));
  }
  std::sort(starts, starts + K);
  for (int32_t i = 0; i < K; ++i) starts[i] += 1 + i * m;
  return GTO_OK;
}

gto_status gto_device_status(gto_ctx* ctx, void* stream, int32_t* host_code) {
  if (!ctx || !host_code) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, ctx->status, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaMemsetAsync(ctx->status, 0, sizeof(word), s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return GTO_ERR_CUDA;
  *host_code = (word & gto::kStatusBadIndex)    ? GTO_ERR_BAD_INDEX
               : (word & gto::kStatusNonFinite) ? GTO_ERR_NONFINITE
                                                : GTO_OK;
  return GTO_OK;
}

int64_t gto_launch_count(const gto_ctx* ctx) { return ctx ? ctx->launches : 0; }

gto_status gto_kernel_timing(gto_ctx* ctx, int enable) {
  if (!ctx) return GTO_ERR_INVALID_ARG;
  ctx->timing = enable != 0;
  return GTO_OK;
}

gto_status gto_kernel_times(gto_ctx* ctx, void* stream, double* total_ms, int64_t* launches) {
  if (!ctx || !total_ms || !launches) return GTO_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return GTO_ERR_CUDA;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return GTO_ERR_CUDA;
  for (int i = 0; i < GTO_K_COUNT; ++i) {
    total_ms[i] = 0.0;
    launches[i] = 0;
  }
  gto_status st = GTO_OK;
  for (size_t i = 0; i < ctx->spans_used; ++i) {
    const gto_ctx::Span& sp = ctx->spans[i];
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, sp.t0, sp.t1) != cudaSuccess) {
      st = GTO_ERR_CUDA;
      continue;
    }
    total_ms[sp.kernel] += ms;
    ++launches[sp.kernel];
  }
  ctx->spans_used = 0;
  return st;
}

}  // extern "C"
