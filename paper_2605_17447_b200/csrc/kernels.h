// Internal launch interface between the C ABI (api.cu) and the kernels. Not installed.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fastocr {

constexpr int kHeadDim = 128;
constexpr int kMaxGroup = 8;          // query heads per KV head handled by one CTA
constexpr int kAttnWarps = 2;         // warps per persistent attention CTA
constexpr int kAttnCtasPerSm = 4;     // resident CTAs per SM (registers and shared memory)
constexpr int kMaxUnits = 512;        // sequences x KV heads per launch (their row prefix lives in shared memory)
constexpr int kMaxPartsPerUnit = 16;  // CTAs sharing one unit in split mode (bounds the last CTA's merge)
constexpr int kMaxGroupLayers = 32;    // consecutive pruned layers one launch can walk (their cache pointers travel in the launch arguments)
constexpr int kMaxGroupCounters = kMaxGroupLayers * kMaxUnits;   // arrival counters: one per (layer of the group, unit)
constexpr int kTopkMaxN = 32768;      // keys of one sequence must fit one CTA's shared memory
constexpr int kTopkMaxHeads = 128;    // query heads the selection kernel can score by itself

// Programmatic dependent launch. Every kernel of this library is launched with the "programmatic
// stream serialization" attribute and (i) lets its successor's CTAs be scheduled as soon as SM
// resources free up (dependents_may_launch), (ii) calls wait_for_prior_grids() before it touches
// anything an earlier kernel may have written or may still be reading; the wait returns when all
// earlier kernels in the stream have completed and their writes are visible. A kernel that has to
// wait before reading some input triggers its successor only after that wait: the successor may
// be told (by the host) that the same input is settled, which is true only from then on. A
// predecessor that is not one of these kernels never triggers early, so ordinary stream order
// applies to it.
#ifdef __CUDACC__
#ifdef FASTOCR_NO_EARLY_LAUNCH   // debug builds: every kernel starts after its predecessor has finished
__device__ __forceinline__ void dependents_may_launch() {}
#else
__device__ __forceinline__ void dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;"); }
#endif
__device__ __forceinline__ void wait_for_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

#ifdef __CUDACC__
// One head's term of a focal score (Section 3.1.1: post-softmax weight, averaged over heads):
// logit and maximum in the log2 domain, inv_sum = 1 / softmax denominator. Heads are added in
// ascending order and the total divided by H; every kernel that forms scores goes through these
// two functions, so that they all produce the same bits.
__device__ __forceinline__ float score_add_head(float acc, float logit, float max_log2, float inv_sum) {
  float e;   // logit <= max: the weight is in (0, 1]; weights below 2^-126 count as 0
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(logit - max_log2));
  return acc + e * inv_sum;
}
__device__ __forceinline__ float score_finish(float acc, int num_q_heads) { return acc / static_cast<float>(num_q_heads); }

// The logits of a focal layer are written with an L2 evict-last policy (they are read back within
// microseconds, while a gigabyte of cache rows streams past) and read with evict-first, so that
// they stop occupying L2 once the scores are formed.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void store_logit(float* dst, float x, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(dst), "f"(x), "l"(policy) : "memory");
}
__device__ __forceinline__ float load_logit(const float* src, uint64_t policy) {
  float x;
  asm volatile("ld.global.cg.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(x) : "l"(src), "l"(policy));
  return x;
}
__device__ __forceinline__ float4 load_logit4(const float* src, uint64_t policy) {
  float4 v;
  asm volatile("ld.global.cg.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(src), "l"(policy));
  return v;
}
#endif

// AttnLaunch::wait_point
constexpr int kWaitBeforeWrites = 0;  // inputs settled long ago: wait only before results / shared workspace are written
constexpr int kWaitAtStart = 1;       // anything may have just been written: wait first
constexpr int kWaitAfterSetup = 2;    // lengths and kept counts are settled, index list / logits workspace are not

struct AttnLaunch {
  // cache view
  const void* k;
  const void* v;              // nullptr: keys only (scores pass)
  int64_t seq_stride_tokens;
  const int32_t* block_table;
  int32_t max_pages;
  int32_t num_pages;          // paged: pages in the pool (block-table entries are clamped to it); 0 = unknown, no check
  int32_t page_size;          // 0 = contiguous; else a power of two
  int32_t page_shift;         // log2(page_size)
  int32_t max_seq_len;        // host bound on seq_len[b] (what the strides / the block table were checked against)
  const int32_t* seq_len;
  const int32_t* vis_start;
  const int32_t* vis_len;
  const uint8_t* seq_mask;    // nullptr, or [B]: only sequences with seq_mask[b] == mask_want take part in this launch
  int32_t mask_want;          //   (the others are neither read nor written: per-sequence focal layer sets)
  int32_t batch, num_q_heads, num_kv_heads;
  float sm_scale;
  const void* q;
  // pruned mode (idx != nullptr)
  const int32_t* idx;
  const int32_t* kcount;
  int32_t k_stride;
  int32_t grid_ctas;          // CTAs launched (kAttnWarps warps each)
  int32_t active_ctas;        // CTAs that take work (<= grid_ctas); the rest exit at once
  int32_t cluster_ctas;       // CTAs per unit when the grid is units x this many and the launch should run one cluster
                              // of that size per unit (a unit's pieces then merge through distributed shared memory); else 0
  int32_t wait_point;         // where the kernel waits for earlier kernels: kWaitAtStart / kWaitAfterSetup / kWaitBeforeWrites
  // A group of consecutive pruned layers in one launch (n_layers > 1; pruned mode only): the layers share
  // lengths, kept counts, index set, block table and geometry and differ in their caches, queries and
  // outputs. The rows of all layers of the group are laid end to end (layer-major) and cut into equal
  // ranges, one per CTA.
  int32_t n_layers;           // 0 or 1: a single layer (k, v, q, out above)
  int64_t q_layer_bytes;      // distance between consecutive layers' queries / outputs
  int64_t out_layer_bytes;
  const void* layer_k[kMaxGroupLayers];
  const void* layer_v[kMaxGroupLayers];
  const int4* plan;           // NULL or one 64-byte record per CTA written by launch_attn_plan for this very launch
                              // shape (grid, lengths, kept counts): the CTA's range and unit, ready made
  // workspace
  float* part_acc;            // [slots][8][128], slot = CTA index + unit index (unit = sequence * Hkv + KV head);
                              // a group launch: slot = 2 x CTA index + (0: the CTA's first piece, 1: its last)
  float* part_ml;             // [slots][8][2]  (max, sum) in the log2 domain
  int32_t* counters;          // [kMaxGroupCounters] arrival counters per (layer of the group, unit), zero between launches
  // results
  void* out;                  // [B][H][128] bf16 or fp32 (unused when v == nullptr)
  int32_t out_is_fp32;
  float* stats;               // nullptr or [B][H][2]: per-head softmax (max, sum) over the whole attended set
  float* logits;              // nullptr or [B][H][n_stride], log2-domain logits of image tokens
  int32_t n_stride;
  unsigned long long* fault_counter;
  unsigned long long* trace;  // debug builds only (FASTOCR_TRACE): per-warp timestamps
};

cudaError_t launch_attn_partial(const AttnLaunch& a, cudaStream_t s);

// Work records for the CTAs of a later launch_attn_partial with the same lengths, kept counts
// and grid (a.grid_ctas): what every CTA would otherwise work out for itself from the lengths of
// all units. plan_out: 4 x int4 per CTA. Several launches may use one plan (the pruned layers of a
// decode step all see the same lengths and the same kept counts).
cudaError_t launch_attn_plan(const AttnLaunch& a, int4* plan_out, cudaStream_t s);

// scores[b][i] = (1/H) sum_h 2^(logit[b][h][i] - max_h) / sum_h  for i < vis_len[b].
cudaError_t launch_scores_finalize(const float* logits, const float* stats, const int32_t* vis_len, int32_t batch,
                                   int32_t num_q_heads, int32_t n_stride_logits, int32_t max_vis_len, float* scores,
                                   int32_t n_stride, cudaStream_t s);

// mass[b] = sum_{i < vis_len[b]} scores[b][i], fixed summation order.
cudaError_t launch_image_mass(const float* scores, int32_t n_stride, const int32_t* vis_len, int32_t batch,
                              float* mass, cudaStream_t s);

// seq_mask: nullptr, or [B]; only sequences with seq_mask[b] == mask_want are selected for (the other rows of
// idx_out are left as they are).
// Scores come either from `scores` ([B][n_stride]) or, when `logits` is not NULL, are formed on the fly
// from the attention kernel's logits ([B][H][n_stride_logits]) and per-head (max, sum) statistics.
cudaError_t launch_select_topk(const float* scores, int32_t n_stride, const int32_t* vis_len, const int32_t* k,
                               int32_t batch, int32_t max_vis_len, int32_t* idx_out, int32_t k_stride,
                               const float* logits, const float* stats, int32_t num_q_heads, int32_t n_stride_logits,
                               cudaStream_t s, const uint8_t* seq_mask = nullptr, int32_t mask_want = 0);

// Kept set of the union variant: out = selected (first selection of a step), current u selected (later
// ones) or current (sequences that are not focal at `layer` when focal_matrix, [L] rows of focal_stride
// entries, is given). Sets are
// ascending index lists [B][stride] with counts [B]; cur_idx may be NULL (nothing to carry over).
cudaError_t launch_union_sets(const int32_t* cur_idx, const int32_t* cur_cnt, int32_t u_stride, const int32_t* sel_idx,
                              const int32_t* sel_cnt, int32_t k_stride, const int32_t* vis_len, int32_t max_vis_len,
                              int32_t batch, int32_t* out_idx, int32_t* out_cnt, const uint8_t* focal_matrix, int32_t layer,
                              int32_t focal_stride, int32_t force_first, int32_t fallback_ran, cudaStream_t s);

cudaError_t configure_kernels();   // one-time cudaFuncSetAttribute calls (current device)

void count_launches(int n);
void count_cluster_launches(int n);   // of those, pruned passes launched as one thread-block cluster per unit

}  // namespace fastocr
