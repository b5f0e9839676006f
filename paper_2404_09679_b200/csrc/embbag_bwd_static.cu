// antdt_embbag_bwd_dedup_static: the backward + dedup step with its scratch inside the library,
// for callers that must not allocate device memory when they run a step (allocator-free serving
// or real-time loops, plug-ins with a memory budget fixed at load time, processes whose device
// memory belongs to another framework's pool).
//
// The scratch is one file-scope __device__ array.  Its name is usable directly in device code,
// but in host code it is only a stand-in symbol, not a device address: handing it to a kernel
// as a pointer would fault (or, where the GPU can reach host memory, silently use the wrong
// memory).  The device address is looked up once per device with cudaGetSymbolAddress while
// that device is current, and that address is what the kernels get.
#include <mutex>

#include "common.cuh"

static __device__ __align__(256) unsigned char g_bwd_scratch[ANTDT_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_ptr[kMaxDevices] = {};
}  // namespace

extern "C" int32_t antdt_embbag_bwd_dedup_static(
    const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets, int64_t n_bags,
    int32_t bags_per_sample, const float* d_pooled, int32_t dim, int64_t n_rows, int32_t n_workers,
    const int64_t* worker_sample_offsets, int32_t* uniq_ids, int64_t* worker_uniq_offsets,
    int64_t* seg_offsets, int32_t* sorted_occ, float* uniq_grads, int64_t out_cap,
    int32_t* dev_status, void* stream) {
  // size check first: nothing is launched for a problem the fixed array cannot hold
  const size_t need = antdt_embbag_bwd_dedup_min_workspace_bytes(nnz, n_bags, dim, n_workers);
  if (need == 0) return ANTDT_ERR_INVALID_ARG;
  if (need > (size_t)ANTDT_STATIC_SCRATCH_BYTES) return ANTDT_ERR_CAPACITY;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ANTDT_ERR_CUDA;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    if (!g_scratch_ptr[dev]) {  // first call on this device: resolve the array's device address
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_bwd_scratch) != cudaSuccess || !p) return ANTDT_ERR_CUDA;
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }
  // The array keeps the previous call's contents.  The shared implementation writes every part
  // of its scratch before reading it and zeroes the one part that is accumulated into (the
  // run-head bit mask) with a memset on the stream, so no extra clearing is needed here.
  return antdt_embbag_bwd_dedup(row_ids, nnz, bag_offsets, n_bags, bags_per_sample, d_pooled, dim,
                                n_rows, n_workers, worker_sample_offsets, uniq_ids,
                                worker_uniq_offsets, seg_offsets, sorted_occ, uniq_grads, out_cap,
                                scratch, (size_t)ANTDT_STATIC_SCRATCH_BYTES, dev_status, stream);
}
