// moga_sort_static: the group sort for callers that cannot hand the library a workspace.
//
// Some hosts of this library may not allocate device memory at the point where they
// need the sort: a plugin called from inside another framework's execution step whose
// memory pool already owns the whole GPU, a service that fixed its device-memory budget
// at start-up, or code that runs where cudaMalloc would synchronise the device in the
// middle of a latency-critical loop.  For them the block histograms and the status word
// the sort kernels need live in the file-scope device array below instead of a caller
// workspace.  The array is part of the library image: every GPU that loads the library
// carries these 1 MiB until the process exits.
#include <mutex>

#include "moga_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;   // 1 MiB: header + B * nblk * M int32 counters
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_sort_scratch[kStaticScratchBytes];

// In host code g_sort_scratch is only a handle for the symbol; the device address has to
// be asked for, per device, with that device current.
std::mutex g_mu;
char* g_scratch_ptr[kMaxDevices] = {nullptr};

moga_status scratch_for_current_device(char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOGA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_sort_scratch) != cudaSuccess || p == nullptr) return MOGA_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return MOGA_OK;
}

}  // namespace

extern "C" moga_status moga_sort_static(const moga_shape* s, const int32_t* gid, int32_t* perm,
                                        int32_t* inv, int32_t* offsets, uint32_t* status_out,
                                        void* stream) {
  if (s == nullptr) return MOGA_ERR_INVALID_ARG;
  // the same shape limits as moga_permute: moga_scratch_bytes is 0 for a shape it rejects
  const size_t need = moga_scratch_bytes(s);
  if (need == 0) return MOGA_ERR_UNSUPPORTED;
  auto ok = [](const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
  if (s->N == 0) {      // no tokens: every group is empty, as in moga_permute; no scratch is touched
    if (!ok(offsets)) return MOGA_ERR_INVALID_ARG;
    MOGA_CUDA_OK(cudaMemsetAsync(offsets, 0, sizeof(int32_t) * s->B * (s->M + 1), static_cast<cudaStream_t>(stream)));
    if (status_out != nullptr) {
      if (reinterpret_cast<uintptr_t>(status_out) & 7u) return MOGA_ERR_INVALID_ARG;
      MOGA_CUDA_OK(cudaMemsetAsync(status_out, 0, 8, static_cast<cudaStream_t>(stream)));
    }
    return MOGA_OK;
  }
  if (!ok(gid) || !ok(perm) || !ok(inv) || !ok(offsets) ||
      (status_out != nullptr && (reinterpret_cast<uintptr_t>(status_out) & 7u)))
    return MOGA_ERR_INVALID_ARG;
  const moga::WsLayout L = moga::ws_layout(*s);
  // Only the header and the histogram block are used; they must fit the static array.
  if (L.sched > kStaticScratchBytes) return MOGA_ERR_WORKSPACE;
  char* scratch = nullptr;
  moga_status st = scratch_for_current_device(&scratch);
  if (st != MOGA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // The array still holds the previous call's words: the status header must start at zero
  // (the histogram block is overwritten in full by the first sort kernel).
  MOGA_CUDA_OK(cudaMemsetAsync(scratch + L.header, 0, 256, cs));
  st = moga::launch_sort(*s, L, gid, perm, inv, offsets, scratch, cs);
  if (st != MOGA_OK) return st;
  if (status_out != nullptr)
    MOGA_CUDA_OK(cudaMemcpyAsync(status_out, scratch + L.header, 8, cudaMemcpyDeviceToDevice, cs));
  return MOGA_OK;
}
