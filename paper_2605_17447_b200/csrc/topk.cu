// TopK of Eq. 2: exact selection of the k best-scored image tokens of every sequence.
//
// Every CTA that works on a sequence holds ALL of the sequence's scores, mapped to order-preserving
// 32-bit keys, in its own shared memory (at most 32768 keys, 128 KB) and selects on its own: the
// key of the k-th largest score is found with a three-pass MSB-first radix select (digits of 11,
// 11 and 10 bits; a pass is a shared-memory histogram and a block-wide scan from the top bin), and
// the result is emitted by an in-order compaction: every key above the threshold, plus the first
// r keys equal to it, where r is what is left of k. Walking the indices in ascending order gives
// both the "lower index wins ties" rule and the ascending output order with no sort.
//
// Given a score array, one CTA per sequence does all of that. In a decode step the scores do not
// exist yet: they are formed here from the focal layer's logits (Section 3.1.1: post-softmax
// weight averaged over the heads), which is the expensive part (H exponentials per token), so a
// thread-block cluster of 1, 2, 4 or 8 CTAs shares it: CTA c scores slice c of the tokens and
// writes the keys into the shared memory of every CTA of the cluster (distributed shared memory);
// after one cluster barrier all CTAs hold the same keys, run the same selection, and CTA c emits
// the selected tokens of slice c. No further communication is needed.
#include "kernels.h"

#include <cooperative_groups.h>

#include <cstdlib>
#include <mutex>

namespace cg = cooperative_groups;

namespace fastocr {
namespace {

#ifdef FASTOCR_TOPK_TRACE
// debug builds: cycle stamps of the selection kernel's phases, 8 per CTA
__device__ long long g_topk_trace[8 * 1024];
__device__ unsigned long long g_topk_wall[2 * 1024];  // wall-clock nanoseconds at entry (after the wait) and at exit
__device__ __forceinline__ unsigned long long topk_wall_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define TOPK_STAMP(i)                                                          \
  do {                                                                         \
    if (threadIdx.x == 0 && blockIdx.x < 1024) {                               \
      g_topk_trace[blockIdx.x * 8 + (i)] = clock64();                          \
      if ((i) == 0) g_topk_wall[blockIdx.x * 2] = topk_wall_now();             \
      if ((i) == 6) g_topk_wall[blockIdx.x * 2 + 1] = topk_wall_now();         \
    }                                                                          \
  } while (0)
#else
#define TOPK_STAMP(i) do { } while (0)
#endif

constexpr int kTopkThreads = 1024;
constexpr int kTopkWarps = kTopkThreads / 32;
constexpr int kTopkMaxCluster = 8;
constexpr int kTopkSplitMinN = 16384;                   // from this many keys on (and >= 4096 per CTA) the selection itself is split over the cluster
constexpr int kTopkBins = 2048;                         // 11-bit digits; two bins per thread
static_assert(kTopkBins == 2 * kTopkThreads, "the bin scan gives every thread two bins");

// larger float <=> larger key; -0 == +0; NaN below everything.
__device__ __forceinline__ uint32_t score_key(float s) {
  if (s != s) return 0u;
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Scores of tokens [lo_i, lo_i + n_loc) of sequence b from a focal layer's logits and per-head
// (max, sum) (Section 3.1.1; the same arithmetic as the stand-alone scoring kernel, head by head in
// ascending order), turned into keys and handed to put1(j, key) / put4(j0, keys[4], count) with j
// relative to lo_i; ready() is called once by every thread, all together, before the first put (the
// place for a barrier that the puts depend on). The logits were written by the kernel just before
// and are read from L2; with `drop_logits` their lines are dropped from L2 afterwards. Every thread
// of the CTA must call this (barriers inside); per_cta is the slice length of the launch (the same
// for every thread).
template <typename Ready, typename Put1, typename Put4>
__device__ __forceinline__ void score_slice(const float* __restrict__ logits, const float* __restrict__ stats, float* head_st,
                                            int b, int num_q_heads, int n_stride_logits, int lo_i, int n_loc, int per_cta,
                                            int drop_logits, Ready ready, Put1 put1, Put4 put4) {
  const int tid = threadIdx.x;
  const float* lp = logits + static_cast<int64_t>(b) * num_q_heads * n_stride_logits + lo_i;
  const uint64_t once = l2_policy_evict_first();
  auto fetch_stats = [&]() {
    for (int i = tid; i < num_q_heads; i += kTopkThreads) {
      head_st[2 * i] = stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2];
      head_st[2 * i + 1] = 1.0f / stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2 + 1];
    }
    __syncthreads();
  };
  if (per_cta <= kTopkThreads) {
    // Few tokens per CTA (small batches, where the kernel is a chain of latencies): one token per
    // thread, up to 32 heads' logits in flight at once, issued before the statistics are fetched.
    const bool live = tid < n_loc;
    float acc = 0.f;
    for (int h0 = 0; h0 < num_q_heads; h0 += 32) {
      float x[32];
#pragma unroll
      for (int j = 0; j < 32; ++j)
        x[j] = (live && h0 + j < num_q_heads) ? load_logit(lp + static_cast<int64_t>(h0 + j) * n_stride_logits + tid, once) : 0.f;
      if (h0 == 0) {
        fetch_stats();
        ready();
      }
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (h0 + j < num_q_heads) acc = score_add_head(acc, x[j], head_st[2 * (h0 + j)], head_st[2 * (h0 + j) + 1]);
    }
    if (live) put1(tid, score_key(score_finish(acc, num_q_heads)));
  } else {
    // four tokens per thread, eight heads' loads in flight
    fetch_stats();
    ready();
    const bool vec = (n_stride_logits & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0;   // lo_i is a multiple of 32
    for (int i0 = tid * 4; i0 < n_loc; i0 += kTopkThreads * 4) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const bool full = vec && i0 + 4 <= n_loc;
      for (int h0 = 0; h0 < num_q_heads; h0 += 8) {
        float4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          x[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (h0 + j < num_q_heads) {
            const float* src = lp + static_cast<int64_t>(h0 + j) * n_stride_logits + i0;
            if (full) {
              x[j] = load_logit4(src, once);
            } else {
              x[j].x = load_logit(src, once);
              if (i0 + 1 < n_loc) x[j].y = load_logit(src + 1, once);
              if (i0 + 2 < n_loc) x[j].z = load_logit(src + 2, once);
              if (i0 + 3 < n_loc) x[j].w = load_logit(src + 3, once);
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (h0 + j < num_q_heads) {
            const float m = head_st[2 * (h0 + j)], inv = head_st[2 * (h0 + j) + 1];
            acc[0] = score_add_head(acc[0], x[j].x, m, inv);
            acc[1] = score_add_head(acc[1], x[j].y, m, inv);
            acc[2] = score_add_head(acc[2], x[j].z, m, inv);
            acc[3] = score_add_head(acc[3], x[j].w, m, inv);
          }
        }
      }
      uint32_t kq[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) kq[j] = score_key(score_finish(acc[j], num_q_heads));
      put4(i0, kq, min(4, n_loc - i0));
    }
  }
  __syncthreads();                                      // every load of this CTA's slice has returned
  if (drop_logits) {
    // The logits are dead now: their lines are dropped from L2 instead of being written back to
    // HBM later, in the middle of the pruned layers' streams (59 MB per focal layer at B = 64,
    // N = 8192). The launch sets the flag only when rows start on 128-byte boundaries; slices
    // are multiples of 32 tokens, so every line here belongs to this CTA alone.
    const int lines = (n_loc + 31) >> 5;
    for (int e = tid; e < num_q_heads * lines; e += kTopkThreads) {
      const int h = e / lines, l = e - h * lines;
      asm volatile("discard.global.L2 [%0], 128;" ::"l"(lp + static_cast<int64_t>(h) * n_stride_logits + 32 * l) : "memory");
    }
  }
}

__global__ void __launch_bounds__(kTopkThreads) select_topk_kernel(const float* __restrict__ scores, int n_stride,
                                                                   const int32_t* __restrict__ vis_len,
                                                                   const int32_t* __restrict__ kreq,
                                                                   int32_t* __restrict__ idx_out, int k_stride, int n_cap,
                                                                   const float* __restrict__ logits,
                                                                   const float* __restrict__ stats, int num_q_heads,
                                                                   int n_stride_logits, int drop_logits,
                                                                   const uint8_t* __restrict__ seq_mask, int mask_want) {
  extern __shared__ __align__(16) uint32_t keys[];      // all keys of the sequence
  __shared__ float head_st[2 * kTopkMaxHeads];          // scoring mode: per head (max, 1 / sum)
  __shared__ uint32_t hist[kTopkBins];
  __shared__ uint32_t hist_first[kTopkBins];            // scoring mode: first-digit histogram of the CTA's own slice, built while scoring
  __shared__ uint32_t warp_gt[kTopkWarps], warp_eq[kTopkWarps];
  __shared__ uint32_t sel_prefix, sel_remaining;

  wait_for_prior_grids();
  dependents_may_launch();
  TOPK_STAMP(0);
  cg::cluster_group cluster = cg::this_cluster();
  const int C = static_cast<int>(cluster.num_blocks());
  const int c = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / C, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = max(min(vis_len[b], n_cap), 0);         // n_cap: what the launch sized the key array for
  int k = kreq[b];
  k = k < 0 ? 0 : (k > N ? N : k);
  k = min(k, k_stride);
  if (seq_mask != nullptr && seq_mask[b] != mask_want) k = 0;   // this sequence's set is not refreshed by this launch
  if (k == 0) return;                                   // the same decision in every CTA of the cluster

  // slice [lo_i, hi_i) of the tokens: what this CTA scores and emits; a multiple of 32 per CTA
  const int per_cta = (((N + C - 1) / C) + 31) & ~31;
  const int lo_i = min(c * per_cta, N), hi_i = min(lo_i + per_cta, N);
  const int n_loc = hi_i - lo_i;
  // A peer's shared memory may be written only once that CTA is known to be running: every CTA
  // signals here and checks for the others just before its first remote store.
  hist[2 * tid] = hist[2 * tid + 1] = 0u;
  hist_first[2 * tid] = hist_first[2 * tid + 1] = 0u;
  if (tid == 0) {
    sel_prefix = 0u;
    sel_remaining = static_cast<uint32_t>(k);
  }
  __syncthreads();                                      // the histograms are clear before anybody counts into them
  if (C > 1) cluster.barrier_arrive();
  if (logits == nullptr) {
    const float* sp = scores + static_cast<int64_t>(b) * n_stride;
    for (int i = tid; i < N; i += kTopkThreads) keys[i] = score_key(sp[i]);
  } else {
    // The CTA scores its slice and writes the keys into every CTA's copy of the key array
    // (distributed shared memory). Before the first remote store all threads, together, make sure
    // that the peers are running (the second half of the barrier begun above).
    // The first radix pass's histogram (top 11 bits) is counted here, key by key as the scores are formed
    // (the threads spend this phase waiting for logits anyway), each CTA for its own slice; the pass itself
    // then only adds up the CTAs' histograms instead of walking all keys.
    auto all_copies = [&](int j, uint32_t key) {
      atomicAdd(&hist_first[key >> 21], 1u);
      for (int r = 0; r < C; ++r) cluster.map_shared_rank(keys, r)[lo_i + j] = key;
    };
    score_slice(logits, stats, head_st, b, num_q_heads, n_stride_logits, lo_i, n_loc, per_cta, drop_logits,
                [&]() {
                  if (C > 1) cluster.barrier_wait();
                },
                all_copies,
                [&](int j0, const uint32_t* kq, int count) {
                  if (count == 4) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) atomicAdd(&hist_first[kq[t] >> 21], 1u);
                    for (int r = 0; r < C; ++r)
                      *reinterpret_cast<uint4*>(cluster.map_shared_rank(keys, r) + lo_i + j0) = make_uint4(kq[0], kq[1], kq[2], kq[3]);
                  } else {
                    for (int t = 0; t < count; ++t) all_copies(j0 + t, kq[t]);
                  }
                });
    TOPK_STAMP(7);
    if (C > 1) cluster.sync();                          // every slice has arrived in every copy
  }
  __syncthreads();
  TOPK_STAMP(1);

  // ---- radix select, three passes over digits of 11, 11 and 10 bits (most significant first) ----
  // Pass p histograms the digit of the keys that match the prefix found so far; thread t then owns
  // bins 2047 - 2t and 2046 - 2t, and a block-wide scan from the top bin finds the digit at which
  // the running count reaches what is left of k.
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const uint32_t digit_mask = pass == 2 ? 0x3ffu : 0x7ffu;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (pass == 1 ? 21 : 10));
    const uint32_t prefix = sel_prefix;
    const uint32_t remaining = sel_remaining;
    const bool counted = pass == 0 && logits != nullptr;   // the first digit was counted while scoring
    for (int base = warp * 32; base < N && !counted; base += kTopkThreads) {   // warp-uniform trip count
      const int i = base + lane;
      const uint32_t key = i < N ? keys[i] : 0u;
      const bool in = i < N && (key & hi_mask) == prefix;
      const uint32_t digit = (key >> shift) & digit_mask;
      if (pass == 0) {
        // the leading bits (sign, exponent) are heavily clustered: aggregate identical digits
        // inside the warp before touching shared memory
        const uint32_t active = __ballot_sync(0xffffffffu, in);
        if (in) {
          const uint32_t peers = __match_any_sync(active, digit);
          if ((__ffs(peers) - 1) == lane) atomicAdd(&hist[digit], __popc(peers));
        }
      } else if (in) {                                  // later digits are spread out and few keys are left
        atomicAdd(&hist[digit], 1u);
      }
    }
    __syncthreads();
    const int d0 = kTopkBins - 1 - 2 * tid, d1 = d0 - 1;   // bins in descending digit order
    uint32_t c0 = hist[d0], c1 = hist[d1];
    hist[d0] = 0u;                                      // ready for the next pass
    hist[d1] = 0u;
    if (counted) {                                      // every CTA of the cluster counted its slice (complete since the barrier above)
      c0 = c1 = 0u;
      for (int r = 0; r < C; ++r) {
        const uint32_t* h = C > 1 ? cluster.map_shared_rank(hist_first, r) : hist_first;
        c0 += h[d0];
        c1 += h[d1];
      }
      if (C > 1) cluster.barrier_arrive();              // (waited for at the end: no CTA leaves while a peer may still read its histogram)
    }
    const uint32_t local = c0 + c1;
    uint32_t incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_gt[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const uint32_t w = warp_gt[lane];
      uint32_t wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += t;
      }
      warp_eq[lane] = wi - w;                           // keys in the warps before this one
    }
    __syncthreads();
    const uint32_t before = warp_eq[warp] + incl - local;   // keys with a larger digit than d0
    if (before < remaining && remaining <= before + local) {   // exactly one thread
      const bool first = before + c0 >= remaining;
      const uint32_t found_digit = first ? d0 : d1;
      sel_prefix = prefix | (found_digit << shift);
      sel_remaining = remaining - (first ? before : before + c0);
    }
    __syncthreads();
    TOPK_STAMP(2 + pass);
  }
  const uint32_t thr = sel_prefix;                      // key of the k-th largest score
  const uint32_t take_eq = sel_remaining;               // how many keys equal to thr are selected

  // ---- in-order compaction over all keys; this CTA emits the tokens of its own slice ------------
  const int per = (N + kTopkThreads - 1) / kTopkThreads;
  const int lo = min(tid * per, N), hi = min(lo + per, N);
  // up to 8 keys per thread (N <= 8192) are kept in registers for the second walk; a full chunk of 8
  // is fetched as two 16-byte loads (a stride of 8 words between lanes would be an 8-way bank conflict)
  constexpr int kRegKeys = 8;
  uint32_t kreg[kRegKeys];
  const bool cached = per <= kRegKeys;
  if (per == kRegKeys && hi - lo == kRegKeys) {
    const uint4 a = *reinterpret_cast<const uint4*>(keys + lo), c4 = *reinterpret_cast<const uint4*>(keys + lo + 4);
    kreg[0] = a.x; kreg[1] = a.y; kreg[2] = a.z; kreg[3] = a.w;
    kreg[4] = c4.x; kreg[5] = c4.y; kreg[6] = c4.z; kreg[7] = c4.w;
  } else if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) kreg[j] = lo + j < hi ? keys[lo + j] : 0u;
  }
  uint32_t gt = 0, eq = 0;
  if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) {
      if (lo + j < hi) {
        gt += kreg[j] > thr;
        eq += kreg[j] == thr;
      }
    }
  }
  // Longer sequences: every warp walks a contiguous region 32 keys at a time (lane = key, no bank
  // conflicts) and counts with ballots; the counts are the same in all lanes of the warp.
  const int per_warp = (((N + kTopkWarps - 1) / kTopkWarps) + 31) & ~31;
  const int w_lo = min(warp * per_warp, N), w_hi = min(w_lo + per_warp, N);
  if (!cached) {
    for (int base = w_lo; base < w_hi; base += 32) {
      const uint32_t key = base + lane < w_hi ? keys[base + lane] : 0u;   // 0 is below every threshold of a non-empty selection
      const bool live = base + lane < w_hi;
      gt += __popc(__ballot_sync(0xffffffffu, live && key > thr));
      eq += __popc(__ballot_sync(0xffffffffu, live && key == thr));
    }
  }
  uint32_t gt_incl = gt, eq_incl = eq;
  if (cached) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t a = __shfl_up_sync(0xffffffffu, gt_incl, o);
      const uint32_t e = __shfl_up_sync(0xffffffffu, eq_incl, o);
      if (lane >= o) {
        gt_incl += a;
        eq_incl += e;
      }
    }
  }
  if (lane == 31) {
    warp_gt[warp] = gt_incl;
    warp_eq[warp] = eq_incl;
  }
  __syncthreads();
  if (warp == 0) {
    uint32_t a = warp_gt[lane], e = warp_eq[lane];
    uint32_t ai = a, ei = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t ta = __shfl_up_sync(0xffffffffu, ai, o);
      const uint32_t te = __shfl_up_sync(0xffffffffu, ei, o);
      if (lane >= o) {
        ai += ta;
        ei += te;
      }
    }
    warp_gt[lane] = ai - a;                             // exclusive
    warp_eq[lane] = ei - e;
  }
  __syncthreads();
  uint32_t gt_before = warp_gt[warp] + gt_incl - gt;
  uint32_t eq_before = warp_eq[warp] + eq_incl - eq;
  TOPK_STAMP(5);
  int32_t* op = idx_out + static_cast<int64_t>(b) * k_stride;
  auto emit = [&](int i, uint32_t key) {
    const bool mine = i >= lo_i && i < hi_i;
    if (key > thr) {
      if (mine) op[gt_before + min(eq_before, take_eq)] = i;
      ++gt_before;
    } else if (key == thr) {
      if (mine && eq_before < take_eq) op[gt_before + eq_before] = i;
      ++eq_before;
    }
  };
  if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j)
      if (lo + j < hi) emit(lo + j, kreg[j]);
  } else {
    const uint32_t below = (1u << lane) - 1u;            // lanes holding lower indices
    uint32_t gt_run = warp_gt[warp], eq_run = warp_eq[warp];
    for (int base = w_lo; base < w_hi; base += 32) {
      const int i = base + lane;
      const bool live = i < w_hi;
      const uint32_t key = live ? keys[i] : 0u;
      const uint32_t m_gt = __ballot_sync(0xffffffffu, live && key > thr);
      const uint32_t m_eq = __ballot_sync(0xffffffffu, live && key == thr);
      gt_before = gt_run + __popc(m_gt & below);
      eq_before = eq_run + __popc(m_eq & below);
      if (live) emit(i, key);
      gt_run += __popc(m_gt);
      eq_run += __popc(m_eq);
    }
  }
  if (C > 1 && logits != nullptr) cluster.barrier_wait();
  TOPK_STAMP(6);
}

// The same selection with the sequence split over the cluster in every phase, for long sequences:
// CTA c scores slice c of the tokens, keeps only that slice's keys, and histograms them; per pass the
// CTAs add up each other's histograms through distributed shared memory (one cluster barrier) and
// all arrive at the same digit; for the compaction every CTA learns how many selected keys the
// slices before its own hold (one more barrier) and emits its slice at that offset. Five cluster
// barriers in all: that pays only when a walk over all keys costs more (N of 16384 and above).
__global__ void __launch_bounds__(kTopkThreads) select_topk_split_kernel(const float* __restrict__ scores, int n_stride,
                                                                   const int32_t* __restrict__ vis_len,
                                                                   const int32_t* __restrict__ kreq,
                                                                   int32_t* __restrict__ idx_out, int k_stride, int n_cap,
                                                                   const float* __restrict__ logits,
                                                                   const float* __restrict__ stats, int num_q_heads,
                                                                   int n_stride_logits, int drop_logits,
                                                                   const uint8_t* __restrict__ seq_mask, int mask_want) {
  extern __shared__ __align__(16) uint32_t keys[];      // keys of the CTA's slice (key of token lo_i + j at j)
  __shared__ float head_st[2 * kTopkMaxHeads];          // scoring mode: per head (max, 1 / sum)
  __shared__ uint32_t hist[2][kTopkBins];               // per pass, alternating: the peers read one while the other refills
  __shared__ uint32_t warp_gt[kTopkWarps], warp_eq[kTopkWarps];
  __shared__ uint32_t sel_prefix, sel_remaining;
  __shared__ uint32_t slice_cnt[2];                     // keys of this slice above / equal to the threshold

  wait_for_prior_grids();
  dependents_may_launch();
  cg::cluster_group cluster = cg::this_cluster();
  const int C = static_cast<int>(cluster.num_blocks());
  const int c = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / C, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = max(min(vis_len[b], n_cap), 0);         // n_cap: what the launch sized the key arrays for
  int k = kreq[b];
  k = k < 0 ? 0 : (k > N ? N : k);
  k = min(k, k_stride);
  if (seq_mask != nullptr && seq_mask[b] != mask_want) k = 0;   // this sequence's set is not refreshed by this launch
  if (k == 0) return;                                   // the same decision in every CTA of the cluster

  // slice [lo_i, hi_i) of the tokens: what this CTA scores, histograms and emits; a multiple of 32 per CTA
  const int per_cta = (((N + C - 1) / C) + 31) & ~31;
  const int lo_i = min(c * per_cta, N), hi_i = min(lo_i + per_cta, N);
  const int n_loc = hi_i - lo_i;
  hist[0][2 * tid] = hist[0][2 * tid + 1] = 0u;
  hist[1][2 * tid] = hist[1][2 * tid + 1] = 0u;
  if (tid == 0) {
    sel_prefix = 0u;
    sel_remaining = static_cast<uint32_t>(k);
  }
  if (logits == nullptr) {
    const float* sp = scores + static_cast<int64_t>(b) * n_stride + lo_i;
    for (int i = tid; i < n_loc; i += kTopkThreads) keys[i] = score_key(sp[i]);
  } else {
    // (the first pass's histogram is counted on the way, as in select_topk_kernel; score_slice has a block
    // barrier between the clearing above and the first key)
    score_slice(logits, stats, head_st, b, num_q_heads, n_stride_logits, lo_i, n_loc, per_cta, drop_logits,
                []() {},
                [&](int j, uint32_t key) {
                  atomicAdd(&hist[0][key >> 21], 1u);
                  keys[j] = key;
                },
                [&](int j0, const uint32_t* kq, int count) {
                  for (int t = 0; t < count; ++t) atomicAdd(&hist[0][kq[t] >> 21], 1u);
                  if (count == 4) {
                    *reinterpret_cast<uint4*>(keys + j0) = make_uint4(kq[0], kq[1], kq[2], kq[3]);
                  } else {
                    for (int t = 0; t < count; ++t) keys[j0 + t] = kq[t];
                  }
                });
  }
  __syncthreads();

  // ---- radix select, three passes over digits of 11, 11 and 10 bits (most significant first) ----
  // Pass p: every CTA histograms the digit of those keys of its slice that match the prefix found so
  // far; after a cluster barrier thread t adds up bins 2047 - 2t and 2046 - 2t of all CTAs' histograms
  // (distributed shared memory), and a block-wide scan from the top bin finds the digit at which the
  // running count reaches what is left of k. Every CTA of the cluster arrives at the same digit.
  for (int pass = 0; pass < 3; ++pass) {
    uint32_t* hb = hist[pass & 1];
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const uint32_t digit_mask = pass == 2 ? 0x3ffu : 0x7ffu;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (pass == 1 ? 21 : 10));
    const uint32_t prefix = sel_prefix;
    const uint32_t remaining = sel_remaining;
    const bool counted = pass == 0 && logits != nullptr;   // the first digit was counted while scoring
    for (int base = warp * 32; base < n_loc && !counted; base += kTopkThreads) {   // warp-uniform trip count
      const int i = base + lane;
      const uint32_t key = i < n_loc ? keys[i] : 0u;
      const bool in = i < n_loc && (key & hi_mask) == prefix;
      const uint32_t digit = (key >> shift) & digit_mask;
      if (pass == 0) {
        // the leading bits (sign, exponent) are heavily clustered: aggregate identical digits
        // inside the warp before touching shared memory
        const uint32_t active = __ballot_sync(0xffffffffu, in);
        if (in) {
          const uint32_t peers = __match_any_sync(active, digit);
          if ((__ffs(peers) - 1) == lane) atomicAdd(&hb[digit], __popc(peers));
        }
      } else if (in) {                                  // later digits are spread out and few keys are left
        atomicAdd(&hb[digit], 1u);
      }
    }
    if (C > 1) cluster.sync(); else __syncthreads();    // every CTA's histogram of this pass is complete
    const int d0 = kTopkBins - 1 - 2 * tid, d1 = d0 - 1;   // bins in descending digit order
    uint32_t c0 = 0u, c1 = 0u;
    if (C > 1) {
      for (int r = 0; r < C; ++r) {
        const uint32_t* h = cluster.map_shared_rank(hb, r);
        c0 += h[d0];
        c1 += h[d1];
      }
    } else {
      c0 = hb[d0];
      c1 = hb[d1];
    }
    // The other histogram is cleared for the next pass: the peers read it in the previous pass, and
    // they were done with that before they arrived at the barrier above.
    hist[(pass + 1) & 1][d0] = 0u;
    hist[(pass + 1) & 1][d1] = 0u;
    const uint32_t local = c0 + c1;
    uint32_t incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_gt[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const uint32_t w = warp_gt[lane];
      uint32_t wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += t;
      }
      warp_eq[lane] = wi - w;                           // keys in the warps before this one
    }
    __syncthreads();
    const uint32_t before = warp_eq[warp] + incl - local;   // keys with a larger digit than d0
    if (before < remaining && remaining <= before + local) {   // exactly one thread
      const bool first = before + c0 >= remaining;
      const uint32_t found_digit = first ? d0 : d1;
      sel_prefix = prefix | (found_digit << shift);
      sel_remaining = remaining - (first ? before : before + c0);
    }
    __syncthreads();
  }
  const uint32_t thr = sel_prefix;                      // key of the k-th largest score
  const uint32_t take_eq = sel_remaining;               // how many keys equal to thr are selected

  // ---- in-order compaction of the CTA's slice ------------------------------------------------------
  const int per = (n_loc + kTopkThreads - 1) / kTopkThreads;
  const int lo = min(tid * per, n_loc), hi = min(lo + per, n_loc);
  // up to 8 keys per thread are kept in registers for the second walk; a full chunk of 8 is fetched
  // as two 16-byte loads (a stride of 8 words between lanes would be an 8-way bank conflict)
  constexpr int kRegKeys = 8;
  uint32_t kreg[kRegKeys];
  const bool cached = per <= kRegKeys;
  if (per == kRegKeys && hi - lo == kRegKeys) {
    const uint4 a = *reinterpret_cast<const uint4*>(keys + lo), c4 = *reinterpret_cast<const uint4*>(keys + lo + 4);
    kreg[0] = a.x; kreg[1] = a.y; kreg[2] = a.z; kreg[3] = a.w;
    kreg[4] = c4.x; kreg[5] = c4.y; kreg[6] = c4.z; kreg[7] = c4.w;
  } else if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) kreg[j] = lo + j < hi ? keys[lo + j] : 0u;
  }
  uint32_t gt = 0, eq = 0;
  if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) {
      if (lo + j < hi) {
        gt += kreg[j] > thr;
        eq += kreg[j] == thr;
      }
    }
  }
  // Longer slices: every warp walks a contiguous region 32 keys at a time (lane = key, no bank
  // conflicts) and counts with ballots; the counts are the same in all lanes of the warp.
  const int per_warp = (((n_loc + kTopkWarps - 1) / kTopkWarps) + 31) & ~31;
  const int w_lo = min(warp * per_warp, n_loc), w_hi = min(w_lo + per_warp, n_loc);
  if (!cached) {
    for (int base = w_lo; base < w_hi; base += 32) {
      const uint32_t key = base + lane < w_hi ? keys[base + lane] : 0u;
      const bool live = base + lane < w_hi;
      gt += __popc(__ballot_sync(0xffffffffu, live && key > thr));
      eq += __popc(__ballot_sync(0xffffffffu, live && key == thr));
    }
  }
  uint32_t gt_incl = gt, eq_incl = eq;
  if (cached) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t a = __shfl_up_sync(0xffffffffu, gt_incl, o);
      const uint32_t e = __shfl_up_sync(0xffffffffu, eq_incl, o);
      if (lane >= o) {
        gt_incl += a;
        eq_incl += e;
      }
    }
  }
  if (lane == 31) {
    warp_gt[warp] = gt_incl;
    warp_eq[warp] = eq_incl;
  }
  __syncthreads();
  if (warp == 0) {
    uint32_t a = warp_gt[lane], e = warp_eq[lane];
    uint32_t ai = a, ei = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t ta = __shfl_up_sync(0xffffffffu, ai, o);
      const uint32_t te = __shfl_up_sync(0xffffffffu, ei, o);
      if (lane >= o) {
        ai += ta;
        ei += te;
      }
    }
    warp_gt[lane] = ai - a;                             // exclusive
    warp_eq[lane] = ei - e;
    if (lane == 31) {
      slice_cnt[0] = ai;                                // the slice's totals, for the CTAs of later slices
      slice_cnt[1] = ei;
    }
  }
  if (C > 1) cluster.sync(); else __syncthreads();
  uint32_t gt_base = 0u, eq_base = 0u;                  // selected keys in the slices before this one
  for (int r = 0; r < c; ++r) {
    const uint32_t* pc = cluster.map_shared_rank(slice_cnt, r);
    gt_base += pc[0];
    eq_base += pc[1];
  }
  uint32_t gt_before = gt_base + warp_gt[warp] + gt_incl - gt;
  uint32_t eq_before = eq_base + warp_eq[warp] + eq_incl - eq;
  int32_t* op = idx_out + static_cast<int64_t>(b) * k_stride;
  auto emit = [&](int j, uint32_t key) {                // key j of the slice = token lo_i + j
    if (key > thr) {
      op[gt_before + min(eq_before, take_eq)] = lo_i + j;
      ++gt_before;
    } else if (key == thr) {
      if (eq_before < take_eq) op[gt_before + eq_before] = lo_i + j;
      ++eq_before;
    }
  };
  if (cached) {
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j)
      if (lo + j < hi) emit(lo + j, kreg[j]);
  } else {
    const uint32_t below = (1u << lane) - 1u;            // lanes holding lower indices
    uint32_t gt_run = gt_base + warp_gt[warp], eq_run = eq_base + warp_eq[warp];
    for (int base = w_lo; base < w_hi; base += 32) {
      const int i = base + lane;
      const bool live = i < w_hi;
      const uint32_t key = live ? keys[i] : 0u;
      const uint32_t m_gt = __ballot_sync(0xffffffffu, live && key > thr);
      const uint32_t m_eq = __ballot_sync(0xffffffffu, live && key == thr);
      gt_before = gt_run + __popc(m_gt & below);
      eq_before = eq_run + __popc(m_eq & below);
      if (live) emit(i, key);
      gt_run += __popc(m_gt);
      eq_run += __popc(m_eq);
    }
  }
  if (C > 1) cluster.sync();                            // no CTA leaves while a peer may still read its counts or histogram
}

}  // namespace

// Clusters of C CTAs with `smem` bytes of dynamic shared memory the device can hold at once; the
// answers are remembered (a handful of distinct shapes per process).
static int max_active_clusters(int C, size_t smem) {
  struct Memo { int c; size_t smem; int n; };
  static Memo memo[16];
  static int used = 0;
  static std::mutex lock;
  std::lock_guard<std::mutex> hold(lock);
  for (int i = 0; i < used; ++i)
    if (memo[i].c == C && memo[i].smem == smem) return memo[i].n;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C);
  cfg.blockDim = dim3(kTopkThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, select_topk_kernel, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    n = 0;
  }
  if (used < 16) memo[used++] = Memo{C, smem, n};
  return n;
}

#ifdef FASTOCR_TOPK_TRACE
extern "C" int fastocr_debug_topk_trace(long long* host_out, int n) {
  return static_cast<int>(cudaMemcpyFromSymbol(host_out, g_topk_trace, sizeof(long long) * n));
}
extern "C" int fastocr_debug_topk_wall(unsigned long long* host_out, int n) {
  return static_cast<int>(cudaMemcpyFromSymbol(host_out, g_topk_wall, sizeof(unsigned long long) * n));
}
#endif

cudaError_t configure_topk() {
  cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkMaxN * 4 + 16);
  if (e != cudaSuccess) return e;
  // same shared-memory carve-out as the attention kernel: no reconfiguration between them
  if ((e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(select_topk_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkMaxN * 4 + 16)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(select_topk_split_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}

cudaError_t launch_select_topk(const float* scores, int32_t n_stride, const int32_t* vis_len, const int32_t* k,
                               int32_t batch, int32_t max_vis_len, int32_t* idx_out, int32_t k_stride,
                               const float* logits, const float* stats, int32_t num_q_heads, int32_t n_stride_logits,
                               cudaStream_t s, const uint8_t* seq_mask, int32_t mask_want) {
  if (batch <= 0 || max_vis_len <= 0) return cudaSuccess;
  if (logits != nullptr && (num_q_heads <= 0 || num_q_heads > kTopkMaxHeads)) return cudaErrorInvalidValue;
  // Cluster size: one CTA per sequence when the scores exist; when they are formed here, enough
  // CTAs to cover the GPU for small batches, with at least 1024 tokens to score per CTA.
  int C = 1;
  if (logits != nullptr) {
    int device = 0, sms = 148;
    if (cudaGetDevice(&device) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    while (C < kTopkMaxCluster && batch * C * 2 <= sms && max_vis_len / (C * 2) >= 1024) C *= 2;
    // all clusters must be resident at once (a second wave doubles the kernel's time): the device says
    // how many clusters of this size and shared-memory footprint it can hold (15 of 8 CTAs on a B200)
    const size_t smem = (static_cast<size_t>(max_vis_len) + 31) / 32 * 32 * 4 + 16;
    while (C > 1 && max_active_clusters(C, smem) < batch) C /= 2;
  }
  // Whole 128-byte lines per (head, 32 tokens): the kernel may drop them from L2 once read. Worth its
  // 2-3 us only when the logits are a load on L2 (tens of MB); small ones are simply overwritten in
  // place by the next focal layer.
  const bool big = static_cast<int64_t>(batch) * num_q_heads * max_vis_len * 4 >= (static_cast<int64_t>(8) << 20);
  const int drop = logits != nullptr && big && (reinterpret_cast<uintptr_t>(logits) & 127) == 0 && (n_stride_logits & 31) == 0 ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(batch * C);
  cfg.blockDim = dim3(kTopkThreads);
  cfg.dynamicSmemBytes = (static_cast<size_t>(max_vis_len) + 31) / 32 * 32 * 4 + 16;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = C;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  static const int split_min_n = [] {                   // tuning knob for experiments, read once
    const char* v = std::getenv("FASTOCR_TOPK_SPLIT_MIN_N");
    return v != nullptr ? std::atoi(v) : kTopkSplitMinN;
  }();
  cudaError_t e;
  // measured: the split variant wins from 16384 keys on when a CTA keeps at least 4096 of them (its five
  // cluster barriers cost about as much as walking 12k keys three times)
  if (C > 1 && max_vis_len >= split_min_n && max_vis_len / C >= 4096) {
    cfg.dynamicSmemBytes = ((static_cast<size_t>(max_vis_len) + C - 1) / C + 31) / 32 * 32 * 4 + 16;   // one slice's keys
    e = cudaLaunchKernelEx(&cfg, select_topk_split_kernel, scores, n_stride, vis_len, k, idx_out, k_stride,
                           static_cast<int>(max_vis_len), logits, stats, static_cast<int>(num_q_heads),
                           static_cast<int>(n_stride_logits), drop, seq_mask, static_cast<int>(mask_want));
  } else {
    e = cudaLaunchKernelEx(&cfg, select_topk_kernel, scores, n_stride, vis_len, k, idx_out, k_stride,
                           static_cast<int>(max_vis_len), logits, stats, static_cast<int>(num_q_heads),
                           static_cast<int>(n_stride_logits), drop, seq_mask, static_cast<int>(mask_want));
  }
  count_launches(1);
  return e;
}

}  // namespace fastocr
