// Kept-set bookkeeping for the variant of the decode step in which the kept image set is the union of
// the focal layers' selections of the current step (Section 3.1.1 speaks of the aggregated set, the
// union over l_i in C of F^t_{l_i}; Algorithm 1 itself replaces the set at every focal layer).
//
// One CTA per sequence. A set is an ascending list of image-token indices (relative to vis_start)
// plus a count. The union of two such lists is formed through a bitmap of the N <= 32768 image
// tokens in shared memory: both lists set their bits, then every thread turns one 32-bit word back
// into indices at the offset a block-wide scan of the words' population counts gives it. The
// output is ascending and free of duplicates by construction.
#include "kernels.h"

namespace fastocr {
namespace {

constexpr int kSetThreads = kTopkMaxN / 32;             // one bitmap word per thread

// What the launch does to sequence b's set:
//   not focal at this layer (per-sequence focal layer sets)          out = current
//   first selection of the step                                      out = selected
//   later selection                                                  out = current u selected
__global__ void __launch_bounds__(kSetThreads) union_sets_kernel(
    const int32_t* __restrict__ cur_idx, const int32_t* __restrict__ cur_cnt, int u_stride,
    const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_cnt, int k_stride,
    const int32_t* __restrict__ vis_len, int n_cap, int32_t* __restrict__ out_idx, int32_t* __restrict__ out_cnt,
    const uint8_t* __restrict__ focal_matrix, int layer, int focal_stride, int force_first, int fallback_ran) {
  __shared__ uint32_t bits[kSetThreads];
  __shared__ uint32_t warp_tot[kSetThreads / 32];
  wait_for_prior_grids();                              // the selection kernel wrote sel_idx just before
  dependents_may_launch();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = max(min(vis_len[b], n_cap), 0);
  const bool focal_here = focal_matrix == nullptr || focal_matrix[static_cast<int64_t>(layer) * focal_stride + b] != 0;
  bool first = force_first != 0;
  if (!first && focal_matrix != nullptr && !fallback_ran) {    // no earlier focal layer of this sequence in this step
    first = true;
    for (int l = 0; l < layer; ++l) first = first && focal_matrix[static_cast<int64_t>(l) * focal_stride + b] == 0;
  }
  const int n_cur = (cur_idx != nullptr && !(focal_here && first)) ? min(max(cur_cnt[b], 0), min(N, u_stride)) : 0;
  const int n_sel = focal_here ? min(max(sel_cnt[b], 0), min(N, k_stride)) : 0;
  bits[tid] = 0u;
  __syncthreads();
  const int32_t* cp = cur_idx != nullptr ? cur_idx + static_cast<int64_t>(b) * u_stride : nullptr;
  const int32_t* sp = sel_idx + static_cast<int64_t>(b) * k_stride;
  for (int i = tid; i < n_cur; i += kSetThreads) {
    const int t = min(max(cp[i], 0), N - 1);
    atomicOr(&bits[t >> 5], 1u << (t & 31));
  }
  for (int i = tid; i < n_sel; i += kSetThreads) {
    const int t = min(max(sp[i], 0), N - 1);
    atomicOr(&bits[t >> 5], 1u << (t & 31));
  }
  __syncthreads();
  uint32_t w = bits[tid];
  const uint32_t mine = __popc(w);
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  uint32_t before = incl - mine, total = 0;
  for (int x = 0; x < kSetThreads / 32; ++x) {
    const uint32_t t = warp_tot[x];
    if (x < warp) before += t;
    total += t;
  }
  int32_t* op = out_idx + static_cast<int64_t>(b) * u_stride;
  while (w != 0u) {
    const int bit = __ffs(w) - 1;
    w &= w - 1;
    if (before < static_cast<uint32_t>(u_stride)) op[before] = tid * 32 + bit;
    ++before;
  }
  if (tid == 0) out_cnt[b] = static_cast<int32_t>(min(total, static_cast<uint32_t>(u_stride)));
}

}  // namespace

cudaError_t launch_union_sets(const int32_t* cur_idx, const int32_t* cur_cnt, int32_t u_stride, const int32_t* sel_idx,
                              const int32_t* sel_cnt, int32_t k_stride, const int32_t* vis_len, int32_t max_vis_len,
                              int32_t batch, int32_t* out_idx, int32_t* out_cnt, const uint8_t* focal_matrix, int32_t layer,
                              int32_t focal_stride, int32_t force_first, int32_t fallback_ran, cudaStream_t s) {
  if (batch <= 0) return cudaSuccess;
  if (max_vis_len > kTopkMaxN) return cudaErrorInvalidValue;
  const cudaError_t e = launch_pdl(union_sets_kernel, dim3(batch), dim3(kSetThreads), 0, s, cur_idx, cur_cnt, u_stride, sel_idx,
                                   sel_cnt, k_stride, vis_len, max_vis_len, out_idx, out_cnt, focal_matrix, layer, focal_stride,
                                   force_first, fallback_ran);
  count_launches(1);
  return e;
}

}  // namespace fastocr
