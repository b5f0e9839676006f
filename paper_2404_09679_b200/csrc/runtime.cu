// Launch accounting, per-kernel CUDA-event timing, the status word reader.
#include <mutex>
#include <string.h>
#include <vector>

#include "common.cuh"

namespace {
struct Slot { const char* name; int64_t launches; double ms; };
struct Pending { int slot; cudaEvent_t a, b; };

std::mutex g_mu;
bool g_profile = false;
thread_local bool t_untimed = false;  // this thread is capturing a stream: no event brackets
int64_t g_launches = 0;
std::vector<Slot> g_slots;
std::vector<Pending> g_pending;
std::vector<cudaEvent_t> g_pool;

cudaEvent_t get_event() {
  if (!g_pool.empty()) {
    cudaEvent_t e = g_pool.back();
    g_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

void drain_locked() {
  for (Pending& p : g_pending) {
    float ms = 0.f;
    if (p.a && p.b && cudaEventSynchronize(p.b) == cudaSuccess &&
        cudaEventElapsedTime(&ms, p.a, p.b) == cudaSuccess) {
      g_slots[p.slot].ms += ms;
    }
    if (p.a) g_pool.push_back(p.a);
    if (p.b) g_pool.push_back(p.b);
  }
  g_pending.clear();
}
}  // namespace

namespace antdt {
namespace {
struct SmallBlob { uint32_t w[512]; };
__global__ void upload_small_kernel(SmallBlob blob, int n_words, uint32_t* dst) {
  for (int i = threadIdx.x; i < n_words; i += blockDim.x) dst[i] = blob.w[i];
}
}  // namespace

// Gather-rate probe: the plainest row gather there is.  A group of `dim/4` lanes owns one output
// row and sums `per_out` input rows picked by consecutive entries of idx, one 16-byte vector per
// lane and row, eight rows requested before the first add.  Timed on a matrix that fits L2 it
// gives the rate at which the SMs can pull scattered rows out of L2, the ceiling of the
// gathering kernels of the step once their rows are cache resident.
template <int G>
__global__ void __launch_bounds__(256)
probe_gather_kernel(const float4* __restrict__ rows, uint32_t n_rows, const int32_t* __restrict__ idx,
                    int64_t n_out, int per_out, float4* __restrict__ out) {
  const int lg = threadIdx.x & (G - 1);
  const int64_t o = ((int64_t)blockIdx.x * 256 + threadIdx.x) / G;
  if (o >= n_out) return;
  const int32_t* my = idx + o * per_out;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < per_out; j0 += 8) {
    float4 v[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const uint32_t r = j0 + t < per_out ? (uint32_t)__ldg(my + j0 + t) : 0u;
      v[t] = __ldg(rows + (size_t)(r < n_rows ? r : 0u) * G + lg);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (j0 + t < per_out) { acc.x += v[t].x; acc.y += v[t].y; acc.z += v[t].z; acc.w += v[t].w; }
    }
  }
  out[o * G + lg] = acc;
}

void upload_small(const void* host, size_t bytes, void* dev, cudaStream_t s) {
  const uint32_t* src = static_cast<const uint32_t*>(host);
  uint32_t* dst = static_cast<uint32_t*>(dev);
  size_t words = bytes / 4;
  while (words > 0) {
    SmallBlob blob;
    const int n = (int)(words < 512 ? words : 512);
    memcpy(blob.w, src, (size_t)n * 4);
    ANTDT_LAUNCH("upload_small", upload_small_kernel, 1, 256, 0, s, blob, n, dst);
    src += n;
    dst += n;
    words -= (size_t)n;
  }
}

int prof_begin(const char* name, cudaStream_t s) {
  std::lock_guard<std::mutex> lk(g_mu);
  ++g_launches;
  if (!g_profile || t_untimed) return -1;
  int slot = -1;
  for (size_t i = 0; i < g_slots.size(); ++i)
    if (g_slots[i].name == name || strcmp(g_slots[i].name, name) == 0) { slot = (int)i; break; }
  if (slot < 0) {
    g_slots.push_back(Slot{name, 0, 0.0});
    slot = (int)g_slots.size() - 1;
  }
  g_slots[slot].launches += 1;
  Pending p{slot, get_event(), get_event()};
  if (p.a) cudaEventRecord(p.a, s);
  g_pending.push_back(p);
  return (int)g_pending.size() - 1;
}

void prof_untimed(bool on) { t_untimed = on; }

void count_launches(int64_t n) {
  std::lock_guard<std::mutex> lk(g_mu);
  g_launches += n;
}

void prof_end(int token, cudaStream_t s) {
  if (token < 0) return;
  std::lock_guard<std::mutex> lk(g_mu);
  if (token < (int)g_pending.size() && g_pending[token].b) cudaEventRecord(g_pending[token].b, s);
}
}  // namespace antdt

extern "C" {

int32_t antdt_read_status(const int32_t* dev_status, void* stream) {
  if (!dev_status) return ANTDT_ERR_INVALID_ARG;
  int32_t h = 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(&h, dev_status, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ANTDT_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return ANTDT_ERR_CUDA;
  return h;
}

int64_t antdt_launch_count(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  return g_launches;
}

int32_t antdt_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> lk(g_mu);
  drain_locked();
  g_slots.clear();
  g_profile = on != 0;
  return ANTDT_OK;
}

int32_t antdt_profile_kernels(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  return (int32_t)g_slots.size();
}

int32_t antdt_profile_get(int32_t idx, char* name, size_t name_cap, int64_t* launches,
                          double* total_ms) {
  std::lock_guard<std::mutex> lk(g_mu);
  drain_locked();
  if (idx < 0 || idx >= (int32_t)g_slots.size()) return ANTDT_ERR_INVALID_ARG;
  if (name && name_cap) {
    strncpy(name, g_slots[idx].name, name_cap - 1);
    name[name_cap - 1] = 0;
  }
  if (launches) *launches = g_slots[idx].launches;
  if (total_ms) *total_ms = g_slots[idx].ms;
  return ANTDT_OK;
}

int32_t antdt_probe_gather(const float* rows, int64_t n_rows, int32_t dim, const int32_t* idx,
                           int64_t n_out, int32_t per_out, float* out, void* stream) {
  if (!rows || !idx || !out || n_rows < 1 || n_rows >= (1ll << 31) || n_out < 0 || per_out < 1 ||
      n_out >= (1ll << 40) / 256)
    return ANTDT_ERR_INVALID_ARG;
  if (!antdt::aligned16(rows) || !antdt::aligned16(out)) return ANTDT_ERR_INVALID_ARG;
  if (n_out == 0) return ANTDT_OK;
  cudaStream_t s = (cudaStream_t)stream;
  const float4* r4 = reinterpret_cast<const float4*>(rows);
  float4* o4 = reinterpret_cast<float4*>(out);
#define PROBE_CASE(G)                                                                            \
  {                                                                                              \
    const unsigned grid = (unsigned)((n_out * G + 255) / 256);                                   \
    ANTDT_LAUNCH("probe_gather", antdt::probe_gather_kernel<G>, grid, 256, 0, s, r4,             \
                 (uint32_t)n_rows, idx, n_out, per_out, o4);                                     \
  }
  if (dim == 16) PROBE_CASE(4)
  else if (dim == 32) PROBE_CASE(8)
  else if (dim == 64) PROBE_CASE(16)
  else if (dim == 128) PROBE_CASE(32)
  else return ANTDT_ERR_INVALID_ARG;
#undef PROBE_CASE
  return antdt::cuda_ok();
}

const char* antdt_version(void) { return "antdt-b200 0.1 (sm_100a)"; }

}  // extern "C"
