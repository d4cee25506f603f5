// TopK of Eq. 2: exact selection of the k best-scored image tokens of every sequence.
//
// One CTA per sequence. The scores are mapped to order-preserving 32-bit keys held in shared
// memory (up to 32768 keys = 128 KB), the key of the k-th largest score is found with a four-pass
// MSB-first radix select (8 bits per pass, 256-bin histogram in shared memory), and the result is
// emitted by an in-order compaction: every key above the threshold, plus the first r keys equal to
// it, where r is what is left of k. Walking the indices in ascending order gives both the
// "lower index wins ties" rule and the ascending output order with no sort.
#include "kernels.h"

namespace fastocr {
namespace {

constexpr int kTopkThreads = 1024;
constexpr int kTopkWarps = kTopkThreads / 32;

// larger float <=> larger key; -0 == +0; NaN below everything.
__device__ __forceinline__ uint32_t score_key(float s) {
  if (s != s) return 0u;
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kTopkThreads) select_topk_kernel(const float* __restrict__ scores, int n_stride,
                                                                   const int32_t* __restrict__ vis_len,
                                                                   const int32_t* __restrict__ kreq,
                                                                   int32_t* __restrict__ idx_out, int k_stride) {
  extern __shared__ uint32_t keys[];                    // [N]
  __shared__ uint32_t hist[256];
  __shared__ uint32_t warp_gt[kTopkWarps], warp_eq[kTopkWarps];
  __shared__ uint32_t sel_prefix, sel_remaining;

  wait_for_prior_grids();
  dependents_may_launch();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = min(vis_len[b], kTopkMaxN);
  int k = kreq[b];
  k = k < 0 ? 0 : (k > N ? N : k);
  k = min(k, k_stride);
  if (k == 0) return;

  const float* sp = scores + static_cast<int64_t>(b) * n_stride;
  for (int i = tid; i < N; i += kTopkThreads) keys[i] = score_key(sp[i]);
  if (tid == 0) {
    sel_prefix = 0u;
    sel_remaining = static_cast<uint32_t>(k);
  }

  // ---- radix select: after pass p the top 8(p+1) bits of the k-th largest key are known -------
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = sel_prefix;
    const uint32_t remaining = sel_remaining;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int base = warp * 32; base < N; base += kTopkThreads) {     // warp-uniform trip count
      const int i = base + lane;
      const uint32_t key = i < N ? keys[i] : 0u;
      const bool in = i < N && (key & hi_mask) == prefix;
      const uint32_t digit = (key >> shift) & 0xffu;
      if (pass == 0) {
        // the leading byte (sign and most of the exponent) is heavily clustered: aggregate
        // identical digits inside the warp before touching shared memory
        const uint32_t active = __ballot_sync(0xffffffffu, in);
        if (in) {
          const uint32_t peers = __match_any_sync(active, digit);
          if ((__ffs(peers) - 1) == lane) atomicAdd(&hist[digit], __popc(peers));
        }
      } else if (in) {                                 // later bytes are spread out and few keys are left
        atomicAdd(&hist[digit], 1u);
      }
    }
    __syncthreads();
    // one warp walks the bins from the top: find the digit where the running count reaches k
    if (warp == 0) {
      uint32_t above = 0;                              // keys with a larger digit
      uint32_t found_digit = 0, found_above = 0;
      bool found = false;
      for (int base = 224; base >= 0 && !found; base -= 32) {
        const uint32_t cnt = hist[base + (31 - lane)]; // lane 0 holds the largest digit of the group
        uint32_t incl = cnt;                           // inclusive scan, largest digit first
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        const bool hit = above + incl >= remaining;
        const uint32_t hits = __ballot_sync(0xffffffffu, hit);
        if (hits) {
          const int src = __ffs(hits) - 1;
          found_digit = base + (31 - src);
          found_above = above + __shfl_sync(0xffffffffu, incl - cnt, src);
          found = true;
        } else {
          above += __shfl_sync(0xffffffffu, incl, 31);
        }
      }
      if (lane == 0) {
        sel_prefix = prefix | (found_digit << shift);
        sel_remaining = remaining - found_above;
      }
    }
    __syncthreads();
  }
  const uint32_t thr = sel_prefix;                      // key of the k-th largest score
  const uint32_t take_eq = sel_remaining;               // how many keys equal to thr are selected

  // ---- in-order compaction --------------------------------------------------------------------
  const int per = (N + kTopkThreads - 1) / kTopkThreads;
  const int lo = min(tid * per, N), hi = min(lo + per, N);
  uint32_t gt = 0, eq = 0;
  for (int i = lo; i < hi; ++i) {
    const uint32_t key = keys[i];
    gt += key > thr;
    eq += key == thr;
  }
  uint32_t gt_incl = gt, eq_incl = eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t a = __shfl_up_sync(0xffffffffu, gt_incl, o);
    const uint32_t c = __shfl_up_sync(0xffffffffu, eq_incl, o);
    if (lane >= o) {
      gt_incl += a;
      eq_incl += c;
    }
  }
  if (lane == 31) {
    warp_gt[warp] = gt_incl;
    warp_eq[warp] = eq_incl;
  }
  __syncthreads();
  if (warp == 0) {
    uint32_t a = warp_gt[lane], c = warp_eq[lane];
    uint32_t ai = a, ci = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t ta = __shfl_up_sync(0xffffffffu, ai, o);
      const uint32_t tc = __shfl_up_sync(0xffffffffu, ci, o);
      if (lane >= o) {
        ai += ta;
        ci += tc;
      }
    }
    warp_gt[lane] = ai - a;                            // exclusive
    warp_eq[lane] = ci - c;
  }
  __syncthreads();
  uint32_t gt_before = warp_gt[warp] + gt_incl - gt;
  uint32_t eq_before = warp_eq[warp] + eq_incl - eq;
  int32_t* op = idx_out + static_cast<int64_t>(b) * k_stride;
  for (int i = lo; i < hi; ++i) {
    const uint32_t key = keys[i];
    if (key > thr) {
      op[gt_before + min(eq_before, take_eq)] = i;
      ++gt_before;
    } else if (key == thr) {
      if (eq_before < take_eq) op[gt_before + eq_before] = i;
      ++eq_before;
    }
  }
}

}  // namespace

cudaError_t configure_topk() {
  cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkMaxN * 4);
  if (e != cudaSuccess) return e;
  // same shared-memory carve-out as the attention kernel: no reconfiguration between them
  return cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}

cudaError_t launch_select_topk(const float* scores, int32_t n_stride, const int32_t* vis_len, const int32_t* k,
                               int32_t batch, int32_t max_vis_len, int32_t* idx_out, int32_t k_stride,
                               cudaStream_t s) {
  if (batch <= 0 || max_vis_len <= 0) return cudaSuccess;
  const cudaError_t e = launch_pdl(select_topk_kernel, dim3(batch), dim3(kTopkThreads), static_cast<size_t>(max_vis_len) * 4, s,
                                   scores, n_stride, vis_len, k, idx_out, k_stride);
  count_launches(1);
  return e;
}

}  // namespace fastocr
