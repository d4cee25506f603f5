// Pruned decode attention for callers that must not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving engine that
// hands every byte of HBM to its own KV-cache pool at start-up, under a framework whose allocator
// must see every allocation, or in a latency-critical decode loop that may not touch the driver's
// allocator at all. fastocr_create allocates a workspace and is therefore unusable for them. The
// entry point below needs no context: the scratch memory of the split merge (per-CTA partial
// results and arrival counters) lives in a fixed-size array that is part of the loaded module.
// The price is a hard size limit and the loss of isolation between calls (see the header).
#include "../../include/fastocr.h"

#include <cmath>
#include <cstdio>
#include <mutex>

#include "kernels.h"

namespace {

constexpr int kNoallocMaxSlots = FASTOCR_NOALLOC_MAX_UNITS + 3 * 160;   // units + persistent CTAs (the launch brings 2 per SM; room for 3 on up to 160 SMs)
constexpr size_t kAccBytes = static_cast<size_t>(kNoallocMaxSlots) * fastocr::kMaxGroup * fastocr::kHeadDim * sizeof(float);
constexpr size_t kMlBytes = static_cast<size_t>(kNoallocMaxSlots) * fastocr::kMaxGroup * 2 * sizeof(float);
constexpr size_t kCounterBytes = static_cast<size_t>(FASTOCR_NOALLOC_MAX_UNITS) * sizeof(int32_t);
constexpr size_t kFaultBytes = 256;
constexpr size_t kScratchBytes = kAccBytes + kMlBytes + kCounterBytes + kFaultBytes;

// The scratch itself: about 3.1 MB held by every GPU that loads the library, until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  int sm_count = 0;
};
constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_lock;              // first calls from several host threads: one of them sets a device up, the others wait
thread_local char g_error[256] = "";

fastocr_status fail(fastocr_status code, const char* msg) {
  snprintf(g_error, sizeof g_error, "%s", msg);
  return code;
}

// Once per device, with that device current: resolve the array's device address (in host code the
// symbol is only a stand-in, not an address a kernel could use) and set the kernels' attributes.
fastocr_status setup_current_device(int device) {
  std::lock_guard<std::mutex> hold(g_setup_lock);     // also orders the fields below for every later caller
  DeviceSetup& s = g_setup[device];
  if (s.ready) return FASTOCR_OK;
  void* ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
  if (e != cudaSuccess || ptr == nullptr) return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));
  int sm = 0;
  if ((e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess)
    return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));
  if ((e = fastocr::configure_kernels()) != cudaSuccess) return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));
  s.scratch = static_cast<unsigned char*>(ptr);
  s.sm_count = sm;
  s.ready = true;
  return FASTOCR_OK;
}

}  // namespace

extern "C" {

const char* fastocr_noalloc_last_error(void) { return g_error; }

int64_t fastocr_noalloc_device_faults(void) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return -1;
  unsigned char* scratch = nullptr;
  {
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (!g_setup[device].ready) return 0;              // no call has run on this device yet
    scratch = g_setup[device].scratch;
  }
  unsigned long long v = 0;
  unsigned char* word = scratch + kAccBytes + kMlBytes + kCounterBytes;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (cudaMemcpy(&v, word, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  if (cudaMemset(word, 0, sizeof v) != cudaSuccess) return -1;
  return static_cast<int64_t>(v);
}

fastocr_status fastocr_sparse_decode_attn_noalloc(const fastocr_kv_view* kv, const void* q, const int32_t* idx,
                                                  const int32_t* k, int32_t k_stride, void* out, int out_is_fp32,
                                                  void* stream) {
  g_error[0] = 0;
  if (kv == nullptr || q == nullptr || idx == nullptr || k == nullptr || out == nullptr)
    return fail(FASTOCR_ERR_INVALID_ARG, "NULL pointer argument");
  if (kv->k == nullptr || kv->v == nullptr || kv->seq_len == nullptr || kv->vis_start == nullptr || kv->vis_len == nullptr)
    return fail(FASTOCR_ERR_INVALID_ARG, "NULL pointer in the cache view");
  if (kv->batch <= 0 || kv->num_q_heads <= 0 || kv->num_kv_heads <= 0 || kv->max_seq_len <= 0 || k_stride <= 0)
    return fail(FASTOCR_ERR_INVALID_ARG, "batch, head counts, max_seq_len and k_stride must be positive");
  if (kv->head_dim != fastocr::kHeadDim) return fail(FASTOCR_ERR_UNSUPPORTED, "head_dim must be 128");
  if (kv->num_q_heads % kv->num_kv_heads != 0) return fail(FASTOCR_ERR_INVALID_ARG, "num_q_heads must be a multiple of num_kv_heads");
  const int G = kv->num_q_heads / kv->num_kv_heads;
  if (G < 1 || G > fastocr::kMaxGroup) return fail(FASTOCR_ERR_UNSUPPORTED, "GQA group size must be 1 to 8");
  if (kv->page_size < 0 || (kv->page_size & (kv->page_size - 1)) != 0) return fail(FASTOCR_ERR_UNSUPPORTED, "page_size must be 0 or a power of two");
  if (kv->page_size > 0 && (kv->block_table == nullptr || static_cast<int64_t>(kv->max_pages) * kv->page_size < kv->max_seq_len))
    return fail(FASTOCR_ERR_INVALID_ARG, "paged view needs a block_table covering max_seq_len");
  if (kv->page_size == 0 && kv->seq_stride_tokens < kv->max_seq_len) return fail(FASTOCR_ERR_INVALID_ARG, "seq_stride_tokens < max_seq_len");
  if (!(kv->sm_scale > 0.f) || !std::isfinite(kv->sm_scale)) return fail(FASTOCR_ERR_INVALID_ARG, "sm_scale must be positive and finite");
  if (kv->page_size > 0 && kv->num_pages < 0) return fail(FASTOCR_ERR_INVALID_ARG, "num_pages must not be negative");
  const int64_t units = static_cast<int64_t>(kv->batch) * kv->num_kv_heads;
  if (units > FASTOCR_NOALLOC_MAX_UNITS) {
    snprintf(g_error, sizeof g_error, "batch x num_kv_heads = %lld exceeds the built-in scratch (limit %d); use a context",
             static_cast<long long>(units), FASTOCR_NOALLOC_MAX_UNITS);
    return FASTOCR_ERR_WORKSPACE;
  }
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));
  if (device < 0 || device >= kMaxDevices) return fail(FASTOCR_ERR_UNSUPPORTED, "device ordinal above 63");
  fastocr_status st = setup_current_device(device);
  if (st != FASTOCR_OK) return st;
  const DeviceSetup& s = g_setup[device];
  // two persistent CTAs per SM (the next launch runs beside them), no idle ones: when every unit
  // gets the same number of CTAs, a grid that is a multiple of the unit count has none left over
  int grid = 2 * s.sm_count;
  if (units <= grid) {
    int parts = grid / static_cast<int>(units);
    if (parts > fastocr::kMaxPartsPerUnit) parts = fastocr::kMaxPartsPerUnit;
    grid = static_cast<int>(units) * parts;
  }
  if (units + grid > kNoallocMaxSlots) return fail(FASTOCR_ERR_WORKSPACE, "this GPU has more SMs than the built-in scratch was sized for");

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // The arrival counters must start at zero; partial slots are written before they are read.
  // (The array keeps whatever the previous call left; the fault word is meant to: it adds up until
  // fastocr_noalloc_device_faults reads and clears it. A module's __device__ arrays start as zeros.)
  unsigned char* counters = s.scratch + kAccBytes + kMlBytes;
  if ((e = cudaMemsetAsync(counters, 0, kCounterBytes, cs)) != cudaSuccess)
    return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));

  fastocr::AttnLaunch a{};
  a.k = kv->k;
  a.v = kv->v;
  a.seq_stride_tokens = kv->seq_stride_tokens;
  a.block_table = kv->block_table;
  a.max_pages = kv->max_pages;
  a.num_pages = kv->page_size > 0 ? kv->num_pages : 0;
  a.max_seq_len = kv->max_seq_len;
  a.page_size = kv->page_size;
  while ((1 << a.page_shift) < kv->page_size) ++a.page_shift;
  a.seq_len = kv->seq_len;
  a.vis_start = kv->vis_start;
  a.vis_len = kv->vis_len;
  a.batch = kv->batch;
  a.num_q_heads = kv->num_q_heads;
  a.num_kv_heads = kv->num_kv_heads;
  a.sm_scale = kv->sm_scale;
  a.q = q;
  a.idx = idx;
  a.kcount = k;
  a.k_stride = k_stride;
  a.grid_ctas = grid;
  a.active_ctas = grid;
  a.wait_point = fastocr::kWaitAtStart;
  a.part_acc = reinterpret_cast<float*>(s.scratch);
  a.part_ml = reinterpret_cast<float*>(s.scratch + kAccBytes);
  a.counters = reinterpret_cast<int32_t*>(counters);
  a.fault_counter = reinterpret_cast<unsigned long long*>(counters + kCounterBytes);
  a.out = out;
  a.out_is_fp32 = out_is_fp32;
  a.stats = nullptr;
  a.logits = nullptr;
  a.trace = nullptr;
  if ((e = fastocr::launch_attn_partial(a, cs)) != cudaSuccess) return fail(FASTOCR_ERR_CUDA, cudaGetErrorString(e));
  return FASTOCR_OK;
}

}  // extern "C"
