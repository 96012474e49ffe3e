// gto_build_tree_noalloc: the tree-building call for callers that may not allocate.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a framework's
// memory-pool discipline where every device byte must come from the framework's allocator,
// in a process that has been handed a fixed memory budget, or on a latency-critical thread
// where an allocation (which can synchronise the whole device) is not acceptable.  For them
// the per-row top-k tables that gto_build_tree keeps in its context's workspace live here in
// a fixed device array that is part of the library image: every GPU that loads the library
// holds these bytes until the process exits.
#include <mutex>

#include "gto_common.cuh"
#include "gto_internal.h"

namespace {

constexpr int64_t kMaxEntries = GTO_NOALLOC_MAX_ENTRIES;  // rows * k
constexpr size_t kIdBytes = kMaxEntries * sizeof(int32_t);
constexpr size_t kZBytes = kMaxEntries * sizeof(float);
constexpr size_t kStatusOffset = kIdBytes + kZBytes;
constexpr size_t kScratchBytes = kStatusOffset + 256;

// Device storage.  In host code this name is only a handle for cudaGetSymbolAddress; the
// device address is looked up once per device below and that pointer goes to the kernels.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};  // device address of g_scratch, per device

struct DeviceScope {
  int prev = -1;
  bool ok;
  explicit DeviceScope(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceScope() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" gto_status gto_build_tree_noalloc(const gto_config* c, int device, const void* draft,
                                             const gto_tree* out, void* stream) {
  if (!c || !draft || !out || !aligned16(draft)) return GTO_ERR_INVALID_ARG;
  {
    const void* const* p = reinterpret_cast<const void* const*>(out);
    for (size_t i = 0; i < sizeof(gto_tree) / sizeof(void*); ++i)
      if (p[i] == nullptr || !aligned16(p[i])) return GTO_ERR_INVALID_ARG;
  }
  if (device < 0 || device >= kMaxDevices) return GTO_ERR_INVALID_ARG;
  if (c->B <= 0 || c->D <= 0 || c->k <= 0 || c->g <= 0 || c->V_draft <= 0)
    return GTO_ERR_INVALID_ARG;
  if (!gto::valid_dtype(c->logit_dtype)) return GTO_ERR_INVALID_ARG;
  if (c->k > c->V_draft) return GTO_ERR_INVALID_ARG;
  const int64_t P = c->k + static_cast<int64_t>(c->D - 1) * c->k * c->k;
  if (c->g > P) return GTO_ERR_INVALID_ARG;
  if (c->G != 2) return GTO_ERR_UNSUPPORTED;
  if (c->k > gto::kMaxTopK || c->k * c->k > gto::kMaxLayer || c->g > gto::kMaxNodes ||
      c->D > gto::kMaxDepth)
    return GTO_ERR_UNSUPPORTED;
  if ((static_cast<int64_t>(c->V_draft) * gto::elem_bytes(c->logit_dtype)) % 16)
    return GTO_ERR_UNSUPPORTED;
  if (static_cast<int64_t>(c->G) * c->B > 65535) return GTO_ERR_UNSUPPORTED;
  const int R = 1 + (c->D - 1) * c->k;
  const int64_t rows = static_cast<int64_t>(c->G) * c->B * R;
  if (rows * c->k > kMaxEntries) return GTO_ERR_TOO_LARGE;  // the fixed scratch cannot hold it

  DeviceScope scope(device);
  if (!scope.ok) return GTO_ERR_CUDA;
  unsigned char* base;
  {
    // first call on this device: resolve the device address of the scratch array
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[device] == nullptr) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || ptr == nullptr) {
        cudaGetLastError();
        return GTO_ERR_CUDA;
      }
      g_scratch_ptr[device] = static_cast<unsigned char*>(ptr);
    }
    base = g_scratch_ptr[device];
  }
  int32_t* top_id = reinterpret_cast<int32_t*>(base);
  float* top_z = reinterpret_cast<float*>(base + kIdBytes);
  int32_t* status = reinterpret_cast<int32_t*>(base + kStatusOffset);

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the status word must start at zero (the
  // top-k tables are fully rewritten for the rows of this call before anything reads them)
  if (cudaMemsetAsync(status, 0, sizeof(int32_t), s) != cudaSuccess) return GTO_ERR_CUDA;
  int64_t launches = 0;
  gto::RowReduceArgs r{};
  r.logits = draft;
  r.dtype = c->logit_dtype;
  r.V = c->V_draft;
  r.R = R;
  r.pad = c->k - 1;
  r.list = nullptr;
  r.list_count = nullptr;
  r.n_rows = static_cast<int>(rows);
  r.k = c->k;
  r.out_lse = out->row_lse;
  r.out_id = top_id;
  r.out_z = top_z;
  r.status = status;
  if (gto::launch_row_reduce(r, s, &launches) != cudaSuccess) return GTO_ERR_CUDA;
  gto::TreeBuildArgs t{};
  t.n_trees = c->G * c->B;
  t.D = c->D;
  t.k = c->k;
  t.g = c->g;
  t.R = R;
  t.row_lse = out->row_lse;
  t.top_id = top_id;
  t.top_z = top_z;
  t.out = *out;
  if (gto::launch_tree_build(t, s, &launches) != cudaSuccess) return GTO_ERR_CUDA;
  return GTO_OK;
}
