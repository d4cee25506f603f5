// C ABI of the FastOCR decode-attention library: context, argument checks, split planning and the
// per-layer / per-step launch sequences. All arithmetic lives in attn.cu and topk.cu.
#include "../../include/fastocr.h"

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "kernels.h"

namespace fastocr {
static std::atomic<long long> g_launches{0};
static std::atomic<long long> g_cluster_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
void count_cluster_launches(int n) { g_cluster_launches.fetch_add(n, std::memory_order_relaxed); }
cudaError_t configure_topk();
}  // namespace fastocr

using fastocr::AttnLaunch;

struct fastocr_ctx {
  int device = 0;
  int sm_count = 148;
  fastocr_limits lim{};
  int64_t cap_items = 0;        // partial slots: one per (team, sequence) pair and KV head
  int4* plan = nullptr;         // launch plan of the decode step's pruned layers: 4 x int4 per CTA
  float* part_acc = nullptr;    // [cap_items][8][128]
  float* part_ml = nullptr;     // [cap_items][8][2]
  int32_t* counters = nullptr;  // [kMaxUnits] arrival counters of the split merge (zero between launches)
  float* logits = nullptr;      // [max_batch][H][max_vis_len]
  float* stats = nullptr;       // [max_batch][H][2]
  float* scores = nullptr;      // [max_batch][max_vis_len] (decode_step scratch)
  int32_t* uni_idx = nullptr;   // [2][max_batch][max_vis_len]: kept image sets of the union variant (current / next)
  int32_t* uni_cnt = nullptr;   // [2][max_batch]
  unsigned long long* faults = nullptr;
  // persistent attention CTAs per SM brought by one launch: a full cache pass takes every slot,
  // a pruned pass half of them (the next layers' launches run beside it; two per SM measured equal
  // to or faster than three on every workload tried, by up to 28 % at 64 units)
  int dense_ctas_per_sm = fastocr::kAttnCtasPerSm;
  int sparse_ctas_per_sm = 2;
  // A pruned launch whose CTAs get at most this many rows each runs a unit's CTAs as one thread-block
  // cluster (merge through distributed shared memory: no global partials, no wait for the previous
  // kernel). Such launches are latency-bound and gain 5-60 %; with more rows per CTA the GPU is full,
  // clusters are harder to place and hold their slots until the slowest CTA is done: 8-13 % slower.
  int cluster_max_rows = 6;
  // Consecutive pruned layers of a decode step that share their lengths and index set run as one launch
  // (up to kMaxGroupLayers of them): its persistent CTAs stream through equal ranges of all those
  // layers' rows, so that layer boundaries cost no launch, no set-up and no pipeline ramp.
  int group_layers = fastocr::kMaxGroupLayers;   // 1 = one launch per layer
  int group_min_rows = 4;                        // rows a CTA of a group launch should have at least
  bool l2_persist_set = false;      // FASTOCR_L2_PERSIST_MB changed the context's persisting-L2 limit: put it back
  size_t l2_persist_before = 0;
  unsigned long long* trace = nullptr;   // set only by debug builds
  unsigned trace_seq = 0;
  char err[512] = {0};
  // optional per-launch timing
  std::vector<cudaEvent_t> prof_ev;   // 2 per timed launch
  std::vector<int> prof_class;
  std::vector<int64_t> prof_count;    // launches covered by each pair
  size_t prof_used = 0;
  bool prof_on = false;
  bool prof_runs = false;             // one pair per run of same-class launches
  bool prof_open = false;
  cudaStream_t prof_stream = nullptr;
};

namespace {

constexpr int kPlanCtas = 4096;   // CTAs a launch plan has room for

fastocr_status fail(fastocr_ctx* ctx, fastocr_status code, const char* fmt, ...) {
  if (ctx != nullptr) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
    va_end(ap);
  }
  return code;
}

bool group_supported(int G) { return G >= 1 && G <= fastocr::kMaxGroup; }

fastocr_status check_view(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, bool need_v) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  if (kv == nullptr || q == nullptr) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL view or query pointer");
  if (kv->k == nullptr || (need_v && kv->v == nullptr)) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL cache pointer");
  if (kv->seq_len == nullptr || kv->vis_start == nullptr || kv->vis_len == nullptr)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL seq_len / vis_start / vis_len");
  if (kv->batch <= 0 || kv->num_q_heads <= 0 || kv->num_kv_heads <= 0 || kv->max_seq_len <= 0)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "batch, head counts and max_seq_len must be positive");
  if (kv->head_dim != fastocr::kHeadDim) return fail(ctx, FASTOCR_ERR_UNSUPPORTED, "head_dim %d (only 128)", kv->head_dim);
  if (kv->num_q_heads % kv->num_kv_heads != 0)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "num_q_heads %d not a multiple of num_kv_heads %d", kv->num_q_heads, kv->num_kv_heads);
  if (!group_supported(kv->num_q_heads / kv->num_kv_heads))
    return fail(ctx, FASTOCR_ERR_UNSUPPORTED, "GQA group size %d (supported: 1 to 8)", kv->num_q_heads / kv->num_kv_heads);
  if (kv->page_size < 0 || (kv->page_size & (kv->page_size - 1)) != 0)
    return fail(ctx, FASTOCR_ERR_UNSUPPORTED, "page_size %d is not 0 or a power of two", kv->page_size);
  if (kv->page_size > 0) {
    if (kv->block_table == nullptr || kv->max_pages <= 0) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "paged view without block_table");
    if (kv->num_pages < 0) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "num_pages must not be negative");
    if (static_cast<int64_t>(kv->max_pages) * kv->page_size < kv->max_seq_len)
      return fail(ctx, FASTOCR_ERR_INVALID_ARG, "max_pages * page_size < max_seq_len");
  } else if (kv->seq_stride_tokens < kv->max_seq_len) {
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "seq_stride_tokens < max_seq_len");
  }
  if (!(kv->sm_scale > 0.f) || !std::isfinite(kv->sm_scale)) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "sm_scale must be positive");
  if (kv->num_kv_heads > fastocr::kMaxUnits)
    return fail(ctx, FASTOCR_ERR_UNSUPPORTED, "num_kv_heads exceeds %d", fastocr::kMaxUnits);
  if (kv->batch > ctx->lim.max_batch || kv->num_q_heads > ctx->lim.num_q_heads ||
      kv->num_kv_heads > ctx->lim.num_kv_heads || kv->max_seq_len > ctx->lim.max_seq_len)
    return fail(ctx, FASTOCR_ERR_WORKSPACE, "view (B=%d H=%d Hkv=%d S<=%d) exceeds the context limits (B=%d H=%d Hkv=%d S<=%d)",
                kv->batch, kv->num_q_heads, kv->num_kv_heads, kv->max_seq_len, ctx->lim.max_batch, ctx->lim.num_q_heads,
                ctx->lim.num_kv_heads, ctx->lim.max_seq_len);
  return FASTOCR_OK;
}

AttnLaunch make_launch(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, bool with_v, int max_len) {
  AttnLaunch a{};
  a.k = kv->k;
  a.v = with_v ? kv->v : nullptr;
  a.seq_stride_tokens = kv->seq_stride_tokens;
  a.block_table = kv->block_table;
  a.max_pages = kv->max_pages;
  a.num_pages = kv->page_size > 0 ? kv->num_pages : 0;
  a.max_seq_len = kv->max_seq_len;
  a.page_size = kv->page_size;
  a.page_shift = 0;
  while ((1 << a.page_shift) < kv->page_size) ++a.page_shift;
  a.seq_len = kv->seq_len;
  a.vis_start = kv->vis_start;
  a.vis_len = kv->vis_len;
  a.batch = kv->batch;
  a.num_q_heads = kv->num_q_heads;
  a.num_kv_heads = kv->num_kv_heads;
  a.sm_scale = kv->sm_scale;
  a.q = q;
  a.part_acc = ctx->part_acc;
  a.part_ml = ctx->part_ml;
  a.fault_counter = ctx->faults;
  a.counters = ctx->counters;
#ifdef FASTOCR_TRACE
  // debug builds: eight rotating trace regions, one per launch
  a.trace = ctx->trace != nullptr ? ctx->trace + (ctx->trace_seq++ % 8) * 32768 : nullptr;
#else
  a.trace = nullptr;
#endif
  a.wait_point = fastocr::kWaitAtStart;
  a.grid_ctas = ctx->sm_count * ctx->dense_ctas_per_sm;
  {
    // small batches: the kernel gives every unit at most kMaxPartsPerUnit CTAs; launch no more
    const int units = kv->batch * kv->num_kv_heads;
    const int64_t rows = static_cast<int64_t>(units) * ((max_len + 31) / 32);
    a.cluster_ctas = 0;
    if (units * fastocr::kMaxPartsPerUnit < a.grid_ctas && rows < static_cast<int64_t>(128) * a.grid_ctas) {
      a.grid_ctas = units * fastocr::kMaxPartsPerUnit;
      // A launch that leaves most SMs empty anyway (a single sequence): one cluster per unit, pieces
      // merged through distributed shared memory. From two sequences on, placing clusters of 16 costs a
      // full-cache pass more than the merge saves (batch 8: 57.6 against 37.3 us).
      if (ctx->cluster_max_rows > 0 && 2 * a.grid_ctas <= ctx->sm_count) a.cluster_ctas = fastocr::kMaxPartsPerUnit;
    }
  }
  a.active_ctas = a.grid_ctas;
  (void)max_len;
  return a;
}

fastocr_status cuda_fail(fastocr_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, FASTOCR_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Brackets launches with events when profiling is on. In per-launch mode every launch gets its own
// event pair (the records between kernels keep consecutive layers from overlapping, so the figures
// are isolated-kernel times including launch latency). In run mode a maximal run of consecutive
// launches of the same class shares one pair: nothing is recorded between them, so they overlap
// exactly as in an unprofiled step, and total time / launches is the in-situ duration.
struct ProfScope {
  fastocr_ctx* ctx;
  cudaStream_t s;
  bool armed = false;
  // n: layers the launch covers (a group launch is timed as that many launches of its class)
  ProfScope(fastocr_ctx* c, int cls, cudaStream_t st, int n = 1) : ctx(c), s(st) {
    if (!c->prof_on) return;
    if (c->prof_runs) {
      if (c->prof_open && c->prof_class.back() == cls) {       // the run goes on
        c->prof_count.back() += n;
        return;
      }
      close_run(c, st);
      if (c->prof_used + 2 > c->prof_ev.size()) return;
      c->prof_class.push_back(cls);
      c->prof_count.push_back(n);
      cudaEventRecord(c->prof_ev[c->prof_used], st);
      c->prof_open = true;
      c->prof_stream = st;
      return;
    }
    if (c->prof_used + 2 <= c->prof_ev.size()) {
      armed = true;
      c->prof_class.push_back(cls);
      c->prof_count.push_back(n);
      cudaEventRecord(c->prof_ev[c->prof_used], st);
    }
  }
  ~ProfScope() {
    if (armed) {
      cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], s);
      ctx->prof_used += 2;
    }
  }
  static void close_run(fastocr_ctx* c, cudaStream_t st) {
    if (!c->prof_open) return;
    cudaEventRecord(c->prof_ev[c->prof_used + 1], st);
    c->prof_used += 2;
    c->prof_open = false;
  }
};

#define FASTOCR_TRY_CUDA(expr, what)                         \
  do {                                                       \
    cudaError_t e_ = (expr);                                 \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_, what);  \
  } while (0)

// One NVTX range per entry point (visible in a timeline when a tool is attached, free otherwise).
struct NvtxScope {
  explicit NvtxScope(const char* name) { nvtxRangePushA(name); }
  ~NvtxScope() { nvtxRangePop(); }
};

// dense pass (+ optional fused scoring) without re-validating the view
// scores_out == NULL with logits_only: logits and per-head statistics are left in the context's
// workspace for a consumer that forms the scores itself (the selection kernel)
fastocr_status dense_impl(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, void* out, int out_is_fp32,
                          float* scores_out, int32_t n_stride, int32_t max_vis, int wait_point, cudaStream_t s,
                          bool logits_only = false, float* image_mass_out = nullptr, const uint8_t* seq_mask = nullptr,
                          int mask_want = 0) {
  AttnLaunch a = make_launch(ctx, kv, q, /*with_v=*/out != nullptr, kv->max_seq_len);
  const bool want_scores = scores_out != nullptr || logits_only;
  if (want_scores) {
    a.logits = ctx->logits;
    a.n_stride = ctx->lim.max_vis_len;
  }
  a.out = out;
  a.out_is_fp32 = out_is_fp32;
  a.wait_point = wait_point;
  a.stats = want_scores ? ctx->stats : nullptr;
  a.seq_mask = seq_mask;
  a.mask_want = mask_want;
  {
    ProfScope p(ctx, out != nullptr ? FASTOCR_PROF_ATTN_DENSE : FASTOCR_PROF_ATTN_KEYS, s);
    FASTOCR_TRY_CUDA(fastocr::launch_attn_partial(a, s), "attention launch");
  }
  if (want_scores && !logits_only) {
    ProfScope p(ctx, FASTOCR_PROF_FINALIZE, s);
    FASTOCR_TRY_CUDA(fastocr::launch_scores_finalize(ctx->logits, ctx->stats, kv->vis_len, kv->batch, kv->num_q_heads,
                                                     ctx->lim.max_vis_len, max_vis, scores_out, n_stride, s),
                     "score finalisation launch");
    if (image_mass_out != nullptr) {
      ProfScope pm(ctx, FASTOCR_PROF_MASS, s);
      FASTOCR_TRY_CUDA(fastocr::launch_image_mass(scores_out, n_stride, kv->vis_len, kv->batch, image_mass_out, s), "image mass launch");
    }
  }
  return FASTOCR_OK;
}

// launch arguments of a pruned pass (everything but the output, the wait point and the plan)
AttnLaunch sparse_args(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, const int32_t* idx, const int32_t* k,
                       int32_t k_stride, int32_t max_kept) {
  const int max_len = (max_kept > 0 && max_kept < kv->max_seq_len) ? max_kept : kv->max_seq_len;
  AttnLaunch a = make_launch(ctx, kv, q, true, max_len);
  a.idx = idx;
  a.kcount = k;
  a.k_stride = k_stride;
  // Leave slots on every SM free for the next layers' launches unless the pass is long enough (per
  // the caller's bound on kept tokens) for the overlap not to matter: then take every slot.
  {
    const int64_t rows = static_cast<int64_t>(kv->batch) * kv->num_kv_heads * ((max_len + 31) / 32);
    const bool long_pass = max_kept > 0 && rows >= static_cast<int64_t>(64) * ctx->sm_count * fastocr::kAttnCtasPerSm;
    a.grid_ctas = ctx->sm_count * (long_pass ? ctx->dense_ctas_per_sm : ctx->sparse_ctas_per_sm);
    // no idle CTAs: when every unit gets the same number of CTAs (the kernel's choice for batches
    // of similar sequences), a grid that is a multiple of the unit count has none left over
    const int units = kv->batch * kv->num_kv_heads;
    if (!long_pass && units <= a.grid_ctas) {
      int parts = a.grid_ctas / units;
      const int max_rows = (max_len + 31) / 32;          // a unit cannot feed more CTAs than it has rows
      if (parts > max_rows) parts = max_rows;
      if (parts > fastocr::kMaxPartsPerUnit) parts = fastocr::kMaxPartsPerUnit;
      a.grid_ctas = units * parts;
      // (parts = what the kernel gives uniform units on this grid)
      if ((max_rows + parts - 1) / parts <= ctx->cluster_max_rows) a.cluster_ctas = parts;
    }
    a.active_ctas = a.grid_ctas;
  }
  return a;
}

// wait_point: how much of this launch may run while earlier kernels of the stream are still
// draining (fastocr::kWait...), i.e. which of its inputs could have been written just before.
// plan: NULL or a launch plan made for exactly these lengths, kept counts and plan_grid CTAs.
fastocr_status sparse_impl(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, const int32_t* idx,
                           const int32_t* k, int32_t k_stride, int32_t max_kept, void* out, int out_is_fp32,
                           int wait_point, cudaStream_t s, const int4* plan = nullptr, int plan_grid = 0,
                           const uint8_t* seq_mask = nullptr, int mask_want = 0) {
  AttnLaunch a = sparse_args(ctx, kv, q, idx, k, k_stride, max_kept);
  a.wait_point = wait_point;
  a.seq_mask = seq_mask;
  a.mask_want = mask_want;
  a.plan = (plan != nullptr && plan_grid == a.grid_ctas) ? plan : nullptr;
  a.out = out;
  a.out_is_fp32 = out_is_fp32;
  {
    ProfScope p(ctx, FASTOCR_PROF_ATTN_SPARSE, s);
    FASTOCR_TRY_CUDA(fastocr::launch_attn_partial(a, s), "attention launch");
  }
  return FASTOCR_OK;
}

// Layers [l0, l0 + n) of a decode step, all pruned over the same index set, as one launch.
fastocr_status group_impl(fastocr_ctx* ctx, const fastocr_kv_view* layers, int n, const void* q, size_t q_bytes, const int32_t* idx,
                          const int32_t* k, int32_t k_stride, int32_t max_kept, void* out, size_t o_bytes, int out_is_fp32,
                          int wait_point, cudaStream_t s) {
  const fastocr_kv_view* kv = &layers[0];
  const int max_len = (max_kept > 0 && max_kept < kv->max_seq_len) ? max_kept : kv->max_seq_len;
  AttnLaunch a = make_launch(ctx, kv, q, true, max_len);
  a.idx = idx;
  a.kcount = k;
  a.k_stride = k_stride;
  a.cluster_ctas = 0;
  a.n_layers = n;
  a.q_layer_bytes = static_cast<int64_t>(q_bytes);
  a.out_layer_bytes = static_cast<int64_t>(o_bytes);
  for (int i = 0; i < n; ++i) {
    a.layer_k[i] = layers[i].k;
    a.layer_v[i] = layers[i].v;
  }
  // every CTA slot of the GPU unless the group is so small that a CTA would get fewer than a few rows
  const int64_t rows = static_cast<int64_t>(kv->batch) * kv->num_kv_heads * ((max_len + 31) / 32) * n;
  int64_t grid = static_cast<int64_t>(ctx->sm_count) * fastocr::kAttnCtasPerSm;
  if (rows < grid * ctx->group_min_rows) grid = rows / ctx->group_min_rows;
  a.grid_ctas = static_cast<int>(grid < 1 ? 1 : grid);
  a.active_ctas = a.grid_ctas;
  a.wait_point = wait_point;
  a.plan = nullptr;
  a.out = out;
  a.out_is_fp32 = out_is_fp32;
  ProfScope p(ctx, FASTOCR_PROF_ATTN_SPARSE, s, n);
  FASTOCR_TRY_CUDA(fastocr::launch_attn_partial(a, s), "attention launch");
  return FASTOCR_OK;
}

// whether two layers' views differ only in their caches (what a group launch requires)
bool same_geometry(const fastocr_kv_view& x, const fastocr_kv_view& y) {
  return x.batch == y.batch && x.num_q_heads == y.num_q_heads && x.num_kv_heads == y.num_kv_heads && x.page_size == y.page_size &&
         x.max_seq_len == y.max_seq_len && x.seq_stride_tokens == y.seq_stride_tokens && x.block_table == y.block_table &&
         x.max_pages == y.max_pages && x.num_pages == y.num_pages && x.seq_len == y.seq_len && x.vis_start == y.vis_start &&
         x.vis_len == y.vis_len && x.sm_scale == y.sm_scale;
}

fastocr_status check_scores_args(fastocr_ctx* ctx, const fastocr_kv_view* kv, const float* scores_out, int32_t n_stride) {
  if (scores_out == nullptr) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL scores_out");
  if (n_stride <= 0) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "n_stride must be positive");
  (void)kv;
  return FASTOCR_OK;
}

// A launch covers at most kMaxUnits (sequence, KV head) pairs: larger batches run as chunks of whole
// sequences, one after the other on the stream (sequences are independent of one another).
int chunk_sequences(const fastocr_kv_view* kv) {
  const int per = fastocr::kMaxUnits / kv->num_kv_heads;
  return kv->batch <= per ? kv->batch : per;
}

// sequences [b0, b0 + nb) of a view
fastocr_kv_view sub_view(const fastocr_kv_view& v, int b0, int nb) {
  fastocr_kv_view s = v;
  s.batch = nb;
  if (v.page_size == 0) {
    const int64_t off = static_cast<int64_t>(b0) * v.seq_stride_tokens * v.num_kv_heads * fastocr::kHeadDim * 2;
    s.k = static_cast<const char*>(v.k) + off;
    if (v.v != nullptr) s.v = static_cast<const char*>(v.v) + off;
  } else {
    s.block_table = v.block_table + static_cast<int64_t>(b0) * v.max_pages;
  }
  s.seq_len = v.seq_len + b0;
  s.vis_start = v.vis_start + b0;
  s.vis_len = v.vis_len + b0;
  return s;
}

}  // namespace

extern "C" {

fastocr_status fastocr_create(fastocr_ctx** out, int device, const fastocr_limits* lim) {
  if (out == nullptr || lim == nullptr) return FASTOCR_ERR_INVALID_ARG;
  *out = nullptr;
  if (lim->max_batch <= 0 || lim->num_q_heads <= 0 || lim->num_kv_heads <= 0 || lim->max_seq_len <= 0 ||
      lim->max_vis_len < 0 || lim->num_q_heads % lim->num_kv_heads != 0)
    return FASTOCR_ERR_INVALID_ARG;
  if (lim->max_vis_len > fastocr::kTopkMaxN) return FASTOCR_ERR_UNSUPPORTED;
  fastocr_ctx* ctx = new (std::nothrow) fastocr_ctx();
  if (ctx == nullptr) return FASTOCR_ERR_WORKSPACE;
  ctx->device = device;
  ctx->lim = *lim;
  cudaError_t e = cudaSetDevice(device);
  int sm = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = fastocr::configure_kernels();
  if (e == cudaSuccess) e = fastocr::configure_topk();
  if (e != cudaSuccess) {
    delete ctx;
    return FASTOCR_ERR_CUDA;
  }
  ctx->sm_count = sm > 0 ? sm : 148;
  // one partial slot per (CTA, unit) pair that can occur: CTAs + units
  if (const char* v = std::getenv("FASTOCR_DENSE_CTAS_PER_SM")) ctx->dense_ctas_per_sm = std::atoi(v);     // tuning knobs,
  if (const char* v = std::getenv("FASTOCR_SPARSE_CTAS_PER_SM")) ctx->sparse_ctas_per_sm = std::atoi(v);   // read once here
  if (const char* v = std::getenv("FASTOCR_CLUSTER_MAX_ROWS")) ctx->cluster_max_rows = std::atoi(v);
  if (const char* v = std::getenv("FASTOCR_GROUP_LAYERS")) ctx->group_layers = std::atoi(v);
  if (const char* v = std::getenv("FASTOCR_GROUP_MIN_ROWS")) ctx->group_min_rows = std::atoi(v);
  if (ctx->group_layers < 1 || ctx->group_layers > fastocr::kMaxGroupLayers) ctx->group_layers = fastocr::kMaxGroupLayers;
  if (ctx->group_min_rows < 1) ctx->group_min_rows = 1;
  if (const char* v = std::getenv("FASTOCR_L2_PERSIST_MB")) {
    // Experiment, off by default: an L2 set-aside for evict-last lines (the logits of a focal layer).
    // It is a limit of this process's CUDA context and takes that much L2 away from everything else.
    int max_persist = 0;
    cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, device);
    size_t want = static_cast<size_t>(std::atoi(v) > 0 ? std::atoi(v) : 0) << 20;
    if (want > static_cast<size_t>(max_persist)) want = static_cast<size_t>(max_persist);
    if (cudaDeviceGetLimit(&ctx->l2_persist_before, cudaLimitPersistingL2CacheSize) == cudaSuccess &&
        cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) == cudaSuccess)
      ctx->l2_persist_set = true;
    (void)cudaGetLastError();
  }
  if (ctx->dense_ctas_per_sm < 1 || ctx->dense_ctas_per_sm > fastocr::kAttnCtasPerSm) ctx->dense_ctas_per_sm = fastocr::kAttnCtasPerSm;
  if (ctx->sparse_ctas_per_sm < 1 || ctx->sparse_ctas_per_sm > fastocr::kAttnCtasPerSm) ctx->sparse_ctas_per_sm = 2;
  // (a group launch uses two slots per CTA instead)
  ctx->cap_items = 2 * static_cast<int64_t>(ctx->sm_count) * fastocr::kAttnCtasPerSm +
                   static_cast<int64_t>(lim->max_batch) * lim->num_kv_heads + 64;
  const int64_t nvis = lim->max_vis_len > 0 ? lim->max_vis_len : 1;
  const size_t bytes_acc = static_cast<size_t>(ctx->cap_items) * fastocr::kMaxGroup * fastocr::kHeadDim * sizeof(float);
  const size_t bytes_ml = static_cast<size_t>(ctx->cap_items) * fastocr::kMaxGroup * 2 * sizeof(float);
  const size_t bytes_logits = static_cast<size_t>(lim->max_batch) * lim->num_q_heads * nvis * sizeof(float);
  const size_t bytes_stats = static_cast<size_t>(lim->max_batch) * lim->num_q_heads * 2 * sizeof(float);
  const size_t bytes_scores = static_cast<size_t>(lim->max_batch) * nvis * sizeof(float);
  if ((e = cudaMalloc(&ctx->part_acc, bytes_acc)) != cudaSuccess || (e = cudaMalloc(&ctx->part_ml, bytes_ml)) != cudaSuccess ||
      (e = cudaMalloc(&ctx->logits, bytes_logits)) != cudaSuccess || (e = cudaMalloc(&ctx->stats, bytes_stats)) != cudaSuccess ||
      (e = cudaMalloc(&ctx->scores, bytes_scores)) != cudaSuccess ||
      (e = cudaMalloc(&ctx->uni_idx, 2 * static_cast<size_t>(lim->max_batch) * nvis * sizeof(int32_t))) != cudaSuccess ||
      (e = cudaMalloc(&ctx->uni_cnt, 2 * static_cast<size_t>(lim->max_batch) * sizeof(int32_t))) != cudaSuccess ||
      (e = cudaMalloc(&ctx->counters, fastocr::kMaxGroupCounters * sizeof(int32_t))) != cudaSuccess ||
      (e = cudaMalloc(&ctx->plan, static_cast<size_t>(kPlanCtas) * 4 * sizeof(int4))) != cudaSuccess ||
      (e = cudaMemset(ctx->counters, 0, fastocr::kMaxGroupCounters * sizeof(int32_t))) != cudaSuccess ||
      (e = cudaMalloc(&ctx->faults, sizeof(unsigned long long))) != cudaSuccess ||
      (e = cudaMemset(ctx->faults, 0, sizeof(unsigned long long))) != cudaSuccess) {
    fastocr_destroy(ctx);
    return e == cudaErrorMemoryAllocation ? FASTOCR_ERR_WORKSPACE : FASTOCR_ERR_CUDA;
  }
  *out = ctx;
  return FASTOCR_OK;
}

void fastocr_destroy(fastocr_ctx* ctx) {
  if (ctx == nullptr) return;
  cudaSetDevice(ctx->device);
  cudaFree(ctx->plan);
  cudaFree(ctx->part_acc);
  cudaFree(ctx->part_ml);
  cudaFree(ctx->logits);
  cudaFree(ctx->stats);
  cudaFree(ctx->scores);
  cudaFree(ctx->uni_idx);
  cudaFree(ctx->uni_cnt);
  cudaFree(ctx->counters);
  cudaFree(ctx->faults);
  if (ctx->l2_persist_set) cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, ctx->l2_persist_before);
  delete ctx;
}

const char* fastocr_last_error(const fastocr_ctx* ctx) { return ctx != nullptr ? ctx->err : "NULL context"; }

int64_t fastocr_device_faults(fastocr_ctx* ctx) {
  if (ctx == nullptr) return -1;
  unsigned long long v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (cudaMemcpy(&v, ctx->faults, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  if (cudaMemset(ctx->faults, 0, sizeof v) != cudaSuccess) return -1;
  return static_cast<int64_t>(v);
}

int32_t fastocr_kept_count(int32_t n_vis, double tau) {
  if (n_vis <= 0 || !(tau > 0.0)) return 0;
  if (tau >= 1.0) return n_vis;
  const double c = std::ceil(tau * static_cast<double>(n_vis) - 1e-9);
  if (c <= 0.0) return 0;
  return c >= static_cast<double>(n_vis) ? n_vis : static_cast<int32_t>(c);
}

fastocr_status fastocr_dense_decode_attn(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, void* out,
                                         int out_is_fp32, float* scores_out, int32_t n_stride, float* image_mass_out,
                                         void* stream) {
  NvtxScope range("fastocr_dense_decode_attn");
  fastocr_status st = check_view(ctx, kv, q, true);
  if (st != FASTOCR_OK) return st;
  if (out == nullptr) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL out");
  int32_t max_vis = 0;
  if (scores_out == nullptr && image_mass_out != nullptr) {      // Eq. 1's ratio alone: the scores go to the context's scratch
    scores_out = ctx->scores;
    n_stride = ctx->lim.max_vis_len;
  }
  if (scores_out != nullptr) {
    if (ctx->lim.max_vis_len <= 0) return fail(ctx, FASTOCR_ERR_WORKSPACE, "context was created with max_vis_len = 0");
    if ((st = check_scores_args(ctx, kv, scores_out, n_stride)) != FASTOCR_OK) return st;
    max_vis = n_stride < ctx->lim.max_vis_len ? n_stride : ctx->lim.max_vis_len;
  }
  const bool scratch_scores = scores_out == ctx->scores;   // every chunk reuses the scratch
  const int64_t per_seq = static_cast<int64_t>(kv->num_q_heads) * fastocr::kHeadDim;
  const int cb = chunk_sequences(kv);
  for (int b0 = 0; b0 < kv->batch; b0 += cb) {
    const fastocr_kv_view sv = sub_view(*kv, b0, kv->batch - b0 < cb ? kv->batch - b0 : cb);
    st = dense_impl(ctx, &sv, static_cast<const char*>(q) + b0 * per_seq * 2, static_cast<char*>(out) + b0 * per_seq * (out_is_fp32 ? 4 : 2),
                    out_is_fp32, (scores_out != nullptr && !scratch_scores) ? scores_out + static_cast<int64_t>(b0) * n_stride : scores_out,
                    n_stride, max_vis, fastocr::kWaitAtStart, static_cast<cudaStream_t>(stream), false,
                    image_mass_out != nullptr ? image_mass_out + b0 : nullptr);
    if (st != FASTOCR_OK) return st;
  }
  return FASTOCR_OK;
}

fastocr_status fastocr_focal_scores(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, float* scores_out,
                                    int32_t n_stride, float* image_mass_out, void* stream) {
  NvtxScope range("fastocr_focal_scores");
  fastocr_status st = check_view(ctx, kv, q, false);
  if (st != FASTOCR_OK) return st;
  if ((st = check_scores_args(ctx, kv, scores_out, n_stride)) != FASTOCR_OK) return st;
  if (ctx->lim.max_vis_len <= 0) return fail(ctx, FASTOCR_ERR_WORKSPACE, "context was created with max_vis_len = 0");
  const int32_t max_vis = n_stride < ctx->lim.max_vis_len ? n_stride : ctx->lim.max_vis_len;
  const int64_t per_seq = static_cast<int64_t>(kv->num_q_heads) * fastocr::kHeadDim;
  const int cb = chunk_sequences(kv);
  for (int b0 = 0; b0 < kv->batch; b0 += cb) {
    const fastocr_kv_view sv = sub_view(*kv, b0, kv->batch - b0 < cb ? kv->batch - b0 : cb);
    st = dense_impl(ctx, &sv, static_cast<const char*>(q) + b0 * per_seq * 2, nullptr, 0, scores_out + static_cast<int64_t>(b0) * n_stride,
                    n_stride, max_vis, fastocr::kWaitAtStart, static_cast<cudaStream_t>(stream), false,
                    image_mass_out != nullptr ? image_mass_out + b0 : nullptr);
    if (st != FASTOCR_OK) return st;
  }
  return FASTOCR_OK;
}

fastocr_status fastocr_select_topk(fastocr_ctx* ctx, const float* scores, int32_t n_stride, const int32_t* vis_len,
                                   const int32_t* k, int32_t batch, int32_t max_vis_len, int32_t* idx_out,
                                   int32_t k_stride, void* stream) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  if (scores == nullptr || vis_len == nullptr || k == nullptr || idx_out == nullptr)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL pointer argument");
  if (batch <= 0 || n_stride <= 0 || k_stride <= 0 || max_vis_len <= 0 || max_vis_len > n_stride)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "need batch, n_stride, k_stride > 0 and 0 < max_vis_len <= n_stride");
  if (max_vis_len > fastocr::kTopkMaxN)
    return fail(ctx, FASTOCR_ERR_UNSUPPORTED, "max_vis_len %d exceeds %d", max_vis_len, fastocr::kTopkMaxN);
  NvtxScope range("fastocr_select_topk");
  ProfScope p(ctx, FASTOCR_PROF_TOPK, static_cast<cudaStream_t>(stream));
  FASTOCR_TRY_CUDA(fastocr::launch_select_topk(scores, n_stride, vis_len, k, batch, max_vis_len, idx_out, k_stride,
                                               nullptr, nullptr, 0, 0, static_cast<cudaStream_t>(stream)),
                   "top-k launch");
  return FASTOCR_OK;
}

fastocr_status fastocr_sparse_decode_attn(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q,
                                          const int32_t* idx, const int32_t* k, int32_t k_stride, int32_t max_kept,
                                          void* out, int out_is_fp32, void* stream) {
  fastocr_status st = check_view(ctx, kv, q, true);
  if (st != FASTOCR_OK) return st;
  if (idx == nullptr || k == nullptr || out == nullptr) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL idx, k or out");
  if (k_stride <= 0 || max_kept < 0) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "k_stride must be positive, max_kept non-negative");
  NvtxScope range("fastocr_sparse_decode_attn");
  const int64_t per_seq = static_cast<int64_t>(kv->num_q_heads) * fastocr::kHeadDim;
  const int cb = chunk_sequences(kv);
  for (int b0 = 0; b0 < kv->batch; b0 += cb) {
    const fastocr_kv_view sv = sub_view(*kv, b0, kv->batch - b0 < cb ? kv->batch - b0 : cb);
    st = sparse_impl(ctx, &sv, static_cast<const char*>(q) + b0 * per_seq * 2, idx + static_cast<int64_t>(b0) * k_stride, k + b0, k_stride,
                     max_kept, static_cast<char*>(out) + b0 * per_seq * (out_is_fp32 ? 4 : 2), out_is_fp32, fastocr::kWaitAtStart,
                     static_cast<cudaStream_t>(stream));
    if (st != FASTOCR_OK) return st;
  }
  return FASTOCR_OK;
}

fastocr_status fastocr_decode_step_ex(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers,
                                      const void* q, void* out, int out_is_fp32, const uint8_t* is_focal,
                                      const int32_t* k, int32_t* fixation, int32_t k_stride, int has_fixation,
                                      int32_t max_vis_len, int32_t max_kept, int* has_fixation_out,
                                      const fastocr_step_options* opt, void* stream) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  const uint8_t* focal_seq = opt != nullptr ? opt->is_focal_seq : nullptr;           // host [L][B]
  const uint8_t* focal_seq_dev = opt != nullptr ? opt->is_focal_seq_dev : nullptr;   // the same on the device
  const bool unite = opt != nullptr && opt->union_sets != 0;
  const fastocr_scores_exchange_fn exchange = opt != nullptr ? opt->scores_exchange : nullptr;
  if (num_layers <= 0 || layers == nullptr || q == nullptr || out == nullptr || (is_focal == nullptr && focal_seq == nullptr) ||
      k == nullptr || fixation == nullptr)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL pointer or num_layers <= 0");
  if ((focal_seq == nullptr) != (focal_seq_dev == nullptr))
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "per-sequence focal sets need both the host and the device copy of the matrix");
  if (k_stride <= 0 || max_vis_len <= 0 || max_vis_len > ctx->lim.max_vis_len)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "k_stride / max_vis_len out of range (context max_vis_len %d)", ctx->lim.max_vis_len);
  for (int l = 0; l < num_layers; ++l) {
    fastocr_status st = check_view(ctx, &layers[l], q, true);
    if (st != FASTOCR_OK) return st;
    if (layers[l].batch != layers[0].batch || layers[l].num_q_heads != layers[0].num_q_heads ||
        layers[l].num_kv_heads != layers[0].num_kv_heads)
      return fail(ctx, FASTOCR_ERR_INVALID_ARG, "layer %d has a different batch / head geometry", l);
  }
  NvtxScope range("fastocr_decode_step");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int B_all = layers[0].batch;
  const int64_t per_seq = static_cast<int64_t>(layers[0].num_q_heads) * fastocr::kHeadDim;
  const size_t q_bytes = B_all * per_seq * 2, o_bytes = B_all * per_seq * (out_is_fp32 ? 4 : 2);   // from one layer to the next
  const int focal_stride = B_all;                      // row length of the per-sequence focal matrix
  // The step over one chunk of the batch (the whole batch unless it has more than kMaxUnits
  // (sequence, KV head) pairs); all arguments are the chunk's own (views, first query / output /
  // index row, first column of the focal matrix).
  auto step_chunk = [&](const fastocr_kv_view* layers, const void* q, void* out, const uint8_t* focal_seq,
                        const uint8_t* focal_seq_dev, const int32_t* k, int32_t* fixation, bool& have_out) -> fastocr_status {
  const int B = layers[0].batch;
  bool have = has_fixation != 0;
  // How many sequences treat layer l as a focal layer: all or none with one focal set for the batch;
  // anything in between with per-sequence sets (Section 3.1.1 profiles C per sample). Layer 0 without
  // a set from the previous step is the fallback: every sequence attends the full cache and selects.
  auto focal_count = [&](int l) {
    if (l == 0 && !have) return B;
    if (focal_seq == nullptr) return is_focal[l] != 0 ? B : 0;
    int n = 0;
    for (int b = 0; b < B; ++b) n += focal_seq[static_cast<size_t>(l) * focal_stride + b] != 0;
    return n;
  };
  // What the launch issued just before the next one was: nothing of this step yet, a pruned or
  // dense attention kernel of this step (it wrote an output slice and the split workspace, neither
  // of which the next attention kernel reads), the selection kernel (it wrote the index set), or
  // the union kernel (it wrote an index set and its counts, on which even the set-up depends).
  enum { kOther, kAttention, kSelection } prev = kOther;
  const bool overlap = !ctx->prof_on || ctx->prof_runs;
  // The kept image set the pruned layers read: Algorithm 1's `fixation` itself, or, in the union
  // variant, one of two buffers of the context that the union kernel fills in turn.
  const int32_t U = ctx->lim.max_vis_len;
  int cur = 0;
  auto uni_idx = [&](int i) { return ctx->uni_idx + static_cast<size_t>(i) * ctx->lim.max_batch * U; };
  auto uni_cnt = [&](int i) { return ctx->uni_cnt + static_cast<size_t>(i) * ctx->lim.max_batch; };
  if (unite && have) {      // what the previous step left is the kept set until this step's first selection
    FASTOCR_TRY_CUDA(fastocr::launch_union_sets(nullptr, nullptr, U, fixation, k, k_stride, layers[0].vis_len, max_vis_len, B,
                                                uni_idx(0), uni_cnt(0), nullptr, 0, focal_stride, 1, 0, s), "kept-set launch");
  }
  // The pruned layers of a step see the same lengths and kept counts: what every CTA of theirs
  // would work out from those (its range, its unit) is computed once, by a small kernel at the
  // head of the step, and handed to each pruned launch as a plan. Layers whose view differs from
  // the first pruned layer's in anything the plan depends on simply run without it, and so do
  // layers that only part of the batch attends pruned, and the union variant (its counts change).
  const fastocr_kv_view* plan_view = nullptr;
  int plan_grid = 0, n_pruned = 0;
  {
    const bool have0 = have;
    for (int l = 0; l < num_layers; ++l) {
      if (focal_count(l) != 0) { have = true; continue; }
      if (plan_view == nullptr) plan_view = &layers[l];
      ++n_pruned;
    }
    have = have0;
  }
  if (n_pruned >= 2 && overlap && !unite && ctx->group_layers == 1) {
    AttnLaunch pa = sparse_args(ctx, plan_view, q, fixation, k, k_stride, max_kept);
    if (pa.grid_ctas <= kPlanCtas) {
      plan_grid = pa.grid_ctas;
      FASTOCR_TRY_CUDA(fastocr::launch_attn_plan(pa, ctx->plan, s), "plan launch");
    }
  }
  auto plan_fits = [&](const fastocr_kv_view& v) {
    return plan_grid > 0 && v.seq_len == plan_view->seq_len && v.vis_start == plan_view->vis_start &&
           v.vis_len == plan_view->vis_len && v.max_seq_len == plan_view->max_seq_len && v.batch == plan_view->batch &&
           v.num_kv_heads == plan_view->num_kv_heads;
  };
  bool selected_this_step = false, fallback_ran = false;
  for (int l = 0; l < num_layers; ++l) {
    const void* ql = static_cast<const char*>(q) + l * q_bytes;
    void* ol = static_cast<char*>(out) + l * o_bytes;
    const int n_focal = focal_count(l);
    const bool fallback = l == 0 && !have;
    const bool mixed = n_focal != 0 && n_focal != B;
    const uint8_t* mask = mixed ? focal_seq_dev + static_cast<size_t>(l) * focal_stride : nullptr;
    fastocr_status st;
    if (n_focal == 0) {
      // a run of layers that the whole batch attends pruned, over the same set and the same lengths: one launch
      int n = 1;
      while (n < ctx->group_layers && l + n < num_layers && focal_count(l + n) == 0 && same_geometry(layers[l], layers[l + n])) ++n;
      const bool fits = static_cast<int64_t>(B) * layers[l].num_kv_heads <= fastocr::kMaxUnits;
      if (n > 1 && overlap && fits) {
        const bool chained = prev != kOther;
        const int wp = !chained ? fastocr::kWaitAtStart : (prev == kAttention ? fastocr::kWaitBeforeWrites : fastocr::kWaitAfterSetup);
        st = group_impl(ctx, &layers[l], n, ql, q_bytes, unite ? uni_idx(cur) : fixation, unite ? uni_cnt(cur) : k,
                        unite ? U : k_stride, max_kept, ol, o_bytes, out_is_fp32, wp, s);
        if (st != FASTOCR_OK) return st;
        prev = kAttention;
        l += n - 1;
        continue;
      }
    }
    if (n_focal != B) {
      // A pruned layer that follows another attention layer reads nothing the latter wrote (its
      // queries, index set and cache were complete before), so the two may overlap; right after
      // a selection only the set-up (lengths, kept counts) may run ahead; after the union kernel
      // (new counts) nothing may.
      const bool chained = prev != kOther && overlap;
      const int wp = !chained ? fastocr::kWaitAtStart : (prev == kAttention ? fastocr::kWaitBeforeWrites : fastocr::kWaitAfterSetup);
      st = sparse_impl(ctx, &layers[l], ql, unite ? uni_idx(cur) : fixation, unite ? uni_cnt(cur) : k, unite ? U : k_stride,
                       max_kept, ol, out_is_fp32, wp, s, (!mixed && plan_fits(layers[l])) ? ctx->plan : nullptr, plan_grid, mask, 0);
      if (st != FASTOCR_OK) return st;
      prev = kAttention;
    }
    if (n_focal != 0) {
      // Full attention + scoring + selection; the refreshed set replaces the current one.
      // The logits workspace is written from the first block on, and its last reader was the
      // previous selection kernel. Right after that kernel the stream must wait for it; once an
      // attention kernel lies in between, that kernel waited for the selection before it let
      // anything else start, so this launch may stream at once, beside the draining pruned pass.
      // The selection kernel forms the scores from the logits itself (no score array, one launch
      // less) unless there are more heads than it has room for, or the scores are to be summed over
      // ranks first (heads sharded over processes).
      const bool chained = prev != kOther && overlap;
      const bool fused = layers[l].num_q_heads <= fastocr::kTopkMaxHeads && exchange == nullptr;
      st = dense_impl(ctx, &layers[l], ql, ol, out_is_fp32, fused ? nullptr : ctx->scores, ctx->lim.max_vis_len, max_vis_len,
                      !chained ? fastocr::kWaitAtStart : (prev == kAttention ? fastocr::kWaitBeforeWrites : fastocr::kWaitAfterSetup),
                      s, fused, nullptr, fallback ? nullptr : mask, 1);
      if (st != FASTOCR_OK) return st;
      if (exchange != nullptr) {
        // heads sharded over processes: the local partial scores are added up over the ranks (the
        // caller's collective, enqueued on this stream) before anything is selected
        if (exchange(ctx->scores, B, ctx->lim.max_vis_len, l, stream, opt->scores_exchange_user) != 0)
          return fail(ctx, FASTOCR_ERR_CUDA, "the scores exchange of layer %d failed", l);
      }
      {
        ProfScope p(ctx, FASTOCR_PROF_TOPK, s);
        FASTOCR_TRY_CUDA(fastocr::launch_select_topk(ctx->scores, ctx->lim.max_vis_len, layers[l].vis_len, k, B,
                                                     max_vis_len, fixation, k_stride, fused ? ctx->logits : nullptr, ctx->stats,
                                                     layers[l].num_q_heads, ctx->lim.max_vis_len, s, fallback ? nullptr : mask, 1),
                         "top-k launch");
      }
      prev = kSelection;
      if (unite) {
        // first selection of the step: the set starts afresh; later ones are added to it
        const int first = (fallback || (focal_seq == nullptr && !selected_this_step)) ? 1 : 0;
        FASTOCR_TRY_CUDA(fastocr::launch_union_sets(uni_idx(cur), uni_cnt(cur), U, fixation, k, k_stride, layers[l].vis_len,
                                                    max_vis_len, B, uni_idx(cur ^ 1), uni_cnt(cur ^ 1),
                                                    fallback ? nullptr : focal_seq_dev, l, focal_stride, first, fallback_ran ? 1 : 0, s),
                         "kept-set launch");
        cur ^= 1;
        prev = kOther;
      }
      if (fallback) fallback_ran = true;
      selected_this_step = true;
      have = true;
    }
  }
  have_out = have;
  return FASTOCR_OK;
  };
  bool have = has_fixation != 0;
  const int cb = chunk_sequences(&layers[0]);
  if (cb >= B_all) {
    const fastocr_status st = step_chunk(layers, q, out, focal_seq, focal_seq_dev, k, fixation, have);
    if (st != FASTOCR_OK) return st;
  } else {
    std::vector<fastocr_kv_view> part(static_cast<size_t>(num_layers));
    for (int b0 = 0; b0 < B_all; b0 += cb) {
      for (int l = 0; l < num_layers; ++l) part[l] = sub_view(layers[l], b0, B_all - b0 < cb ? B_all - b0 : cb);
      const fastocr_status st = step_chunk(part.data(), static_cast<const char*>(q) + b0 * per_seq * 2,
                                           static_cast<char*>(out) + b0 * per_seq * (out_is_fp32 ? 4 : 2),
                                           focal_seq != nullptr ? focal_seq + b0 : nullptr,
                                           focal_seq_dev != nullptr ? focal_seq_dev + b0 : nullptr, k + b0,
                                           fixation + static_cast<int64_t>(b0) * k_stride, have);
      if (st != FASTOCR_OK) return st;
    }
  }
  if (has_fixation_out != nullptr) *has_fixation_out = have ? 1 : 0;
  return FASTOCR_OK;
}

fastocr_status fastocr_decode_step(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers,
                                   const void* q, void* out, int out_is_fp32, const uint8_t* is_focal,
                                   const int32_t* k, int32_t* fixation, int32_t k_stride, int has_fixation,
                                   int32_t max_vis_len, int32_t max_kept, int* has_fixation_out, void* stream) {
  return fastocr_decode_step_ex(ctx, num_layers, layers, q, out, out_is_fp32, is_focal, k, fixation, k_stride, has_fixation,
                                max_vis_len, max_kept, has_fixation_out, nullptr, stream);
}

fastocr_status fastocr_warmup_step(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers, const void* q,
                                   void* out, int out_is_fp32, float* ratio_out, void* stream) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  if (num_layers <= 0 || layers == nullptr || q == nullptr || out == nullptr || ratio_out == nullptr)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "NULL pointer or num_layers <= 0");
  if (ctx->lim.max_vis_len <= 0) return fail(ctx, FASTOCR_ERR_WORKSPACE, "context was created with max_vis_len = 0");
  for (int l = 0; l < num_layers; ++l) {
    fastocr_status st = check_view(ctx, &layers[l], q, true);
    if (st != FASTOCR_OK) return st;
    if (layers[l].batch != layers[0].batch || layers[l].num_q_heads != layers[0].num_q_heads)
      return fail(ctx, FASTOCR_ERR_INVALID_ARG, "layer %d has a different batch / head geometry", l);
  }
  NvtxScope range("fastocr_warmup_step");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int B = layers[0].batch;
  const int64_t per_layer = static_cast<int64_t>(B) * layers[0].num_q_heads * fastocr::kHeadDim;
  const size_t q_bytes = per_layer * 2, o_bytes = per_layer * (out_is_fp32 ? 4 : 2);
  const int64_t per_seq = static_cast<int64_t>(layers[0].num_q_heads) * fastocr::kHeadDim;
  const int cb = chunk_sequences(&layers[0]);
  for (int l = 0; l < num_layers; ++l) {
    // one pass over K and V: the layer's output, and from the same logits the head-averaged image
    // attention whose sum over the image span is Eq. 1's ratio (batches beyond a launch's reach: in chunks)
    for (int b0 = 0; b0 < B; b0 += cb) {
      const fastocr_kv_view sv = sub_view(layers[l], b0, B - b0 < cb ? B - b0 : cb);
      fastocr_status st = dense_impl(ctx, &sv, static_cast<const char*>(q) + l * q_bytes + b0 * per_seq * 2,
                                     static_cast<char*>(out) + l * o_bytes + b0 * per_seq * (out_is_fp32 ? 4 : 2), out_is_fp32, ctx->scores,
                                     ctx->lim.max_vis_len, ctx->lim.max_vis_len, fastocr::kWaitAtStart, s, false,
                                     ratio_out + static_cast<size_t>(l) * B + b0);
      if (st != FASTOCR_OK) return st;
    }
  }
  return FASTOCR_OK;
}

int32_t fastocr_focal_layers(const double* mean_ratio, int32_t num_layers, double rho, int32_t gap, int32_t* focal_out) {
  if (mean_ratio == nullptr || focal_out == nullptr || num_layers <= 0 || gap < 0 || !(rho >= 0.0)) return -1;
  const int budget = static_cast<int>(std::floor(rho * num_layers + 1e-9));
  std::vector<char> used(num_layers, 0), chosen(num_layers, 0);
  int count = 0;
  // walk the layers from the highest mean ratio down (selection sort keeps ties in layer order)
  for (int step = 0; step < num_layers && count < budget; ++step) {
    int best = -1;
    for (int l = 0; l < num_layers; ++l)
      if (!used[l] && (best < 0 || mean_ratio[l] > mean_ratio[best])) best = l;
    used[best] = 1;
    bool far_enough = true;
    for (int l = 0; l < num_layers; ++l)
      if (chosen[l] && std::abs(l - best) <= gap) far_enough = false;
    if (far_enough) {
      chosen[best] = 1;
      ++count;
    }
  }
  int n = 0;
  for (int l = 0; l < num_layers; ++l)
    if (chosen[l]) focal_out[n++] = l;
  return n;
}

double fastocr_attn_flops(double batch, double layers, double hidden, double seq_len) {
  return batch * layers * (8.0 * hidden * hidden + 4.0 * hidden * seq_len);
}

double fastocr_attn_flops_pruned(double batch, double layers, double hidden, double seq_len, double full_layers,
                                 double kept_len) {
  const double proj = 8.0 * hidden * hidden * layers;                    // every layer projects the new token
  const double attend = 4.0 * hidden * (full_layers * seq_len + (layers - full_layers) * kept_len);
  return batch * (proj + attend);
}

fastocr_status fastocr_profile_begin(fastocr_ctx* ctx, int32_t max_launches, int coalesce_runs) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  if (max_launches <= 0 || ctx->prof_on) return fail(ctx, FASTOCR_ERR_INVALID_ARG, "profile_begin: bad size or already profiling");
  cudaSetDevice(ctx->device);
  ctx->prof_ev.assign(static_cast<size_t>(max_launches) * 2, nullptr);
  for (auto& ev : ctx->prof_ev) FASTOCR_TRY_CUDA(cudaEventCreate(&ev), "cudaEventCreate");
  ctx->prof_class.clear();
  ctx->prof_class.reserve(max_launches);
  ctx->prof_count.clear();
  ctx->prof_count.reserve(max_launches);
  ctx->prof_used = 0;
  ctx->prof_runs = coalesce_runs != 0;
  ctx->prof_open = false;
  ctx->prof_on = true;
  return FASTOCR_OK;
}

fastocr_status fastocr_profile_end(fastocr_ctx* ctx, double* ms_per_class, int64_t* launches_per_class) {
  if (ctx == nullptr) return FASTOCR_ERR_INVALID_ARG;
  if (!ctx->prof_on || ms_per_class == nullptr || launches_per_class == nullptr)
    return fail(ctx, FASTOCR_ERR_INVALID_ARG, "profile_end: not profiling or NULL output");
  ProfScope::close_run(ctx, ctx->prof_stream);
  ctx->prof_on = false;
  for (int c = 0; c < FASTOCR_PROF_CLASSES; ++c) {
    ms_per_class[c] = 0.0;
    launches_per_class[c] = 0;
  }
  cudaError_t e = cudaDeviceSynchronize();
  for (size_t i = 0; e == cudaSuccess && i + 2 <= ctx->prof_used && i / 2 < ctx->prof_class.size(); i += 2) {
    float ms = 0.f;
    e = cudaEventElapsedTime(&ms, ctx->prof_ev[i], ctx->prof_ev[i + 1]);
    ms_per_class[ctx->prof_class[i / 2]] += ms;
    launches_per_class[ctx->prof_class[i / 2]] += ctx->prof_count[i / 2];
  }
  for (auto ev : ctx->prof_ev) cudaEventDestroy(ev);
  ctx->prof_ev.clear();
  ctx->prof_class.clear();
  ctx->prof_count.clear();
  ctx->prof_used = 0;
  if (e != cudaSuccess) return cuda_fail(ctx, e, "profile_end");
  return FASTOCR_OK;
}

#ifdef FASTOCR_TRACE
// debug builds: device buffer of 8 timestamps per attention warp (not part of the public interface)
void fastocr_debug_set_trace(fastocr_ctx* ctx, unsigned long long* buf) { ctx->trace = buf; }
#endif

int64_t fastocr_launch_count(void) { return fastocr::g_launches.load(std::memory_order_relaxed); }
int64_t fastocr_cluster_launch_count(void) { return fastocr::g_cluster_launches.load(std::memory_order_relaxed); }

}  // extern "C"
