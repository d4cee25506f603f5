// Decode attention kernels for sm_100a: one templated persistent flash-decode core serves dense
// attention (Eq. 2, focal case), the keys-only scoring pass, and pruned attention over the kept
// set K = T u F (Eq. 2, non-focal case), on contiguous or paged caches.
//
// Work decomposition (stream-K over tokens). A unit is one (sequence, KV head) pair; its attended
// tokens are cut into rows of 32 (one 16-token block per warp of a CTA). The rows of the launch
// are divided among persistent CTAs of two warps: equal parts of every unit when the units are of
// similar length and no more numerous than the CTAs (no CTA then straddles two units), else
// equal ranges of all rows laid end to end. Four CTAs fit an SM; a full-cache pass brings all four,
// a pruned pass two, so that the next layers' launches (which start early through programmatic
// dependent launch) can run beside it. Every CTA streams about the same number of
// rows, pays one pipeline prologue per unit piece and exits without waiting for anyone. When a
// CTA leaves a unit, its warps merge their running (max, sum, output) through a 4 KB shared-memory
// buffer; a unit held by one CTA is normalised and written at once, a unit shared by several CTAs
// goes through global partials and is merged by whichever CTA arrives last (one atomic arrival
// counter per unit, no spinning), or, for passes launched with one thread-block cluster per unit
// (short pruned passes, full-cache passes of small batches), is merged by the cluster's first CTA
// out of the others' shared memory (no global traffic, so no waiting for the previous kernel either). How the rows are handed out is worked out by every CTA from the
// lengths of all units (one round trip, a scan) or, for the pruned layers of a decode step, which
// all see the same lengths and kept counts, once per step by attn_plan_kernel: a CTA then reads a
// 64-byte record with its range, its unit and the unit's geometry.
//
// Data path: a block's 16 K rows and 16 V rows (256 bytes each) travel HBM -> shared memory with
// 16-byte cp.async (marked evict-first in L2: cache rows are read once per layer), one full row
// per half-warp per instruction (so every request covers whole 128-byte lines), into a per-warp
// ring of kStages blocks (hand-off inside the warp only: __syncwarp). The K tile and the V tile of
// a block are separate copy groups: K is waited for at the top of the block's iteration, V only
// after the softmax, and the copies of the block kDepth ahead go out as soon as a tile's fragments
// are in registers (K) or while the tensor cores work (V). kDepth is 3 for pruned passes (more
// latency hidden per warp) and 2 for full-cache passes (which saturate HBM anyway and run faster
// with fewer requests queued). Rows are stored with their 16-byte chunks XOR-swizzled by the token's
// low three bits so that ldmatrix reads are bank-conflict free. Cache rows are located ahead of
// the copies by lanes 0-15 (one token each): first the logical position (a load from the index
// list for selected image tokens), one block later the physical row (a block-table load for paged
// caches), one block later the copy, so neither lookup sits on the critical path; when a segment
// starts, the lookups of its first blocks are issued together. A pruned pass also touches one line
// in every 2 MiB page of its sequence's cache span at once: the address-translation misses that
// random rows would otherwise take one by one in mid-stream are then taken in parallel. A CTA
// whose range covers pieces of several units handles them one after the other, refilling the
// pipeline at each boundary.
//
// Arithmetic: with a GQA group of 7 or 8 query heads per KV head, q.K^T and P.V are skinny matrix
// products ([16 tokens x 128] x [128 x 8 heads]); on the fp32 CUDA cores they need more issue slots
// than the HBM stream leaves time for, so both run on the tensor cores as warp-level
// mma.sync.m16n8k16 (bf16 inputs, fp32 accumulation):
//   S[token][head]  = K[token][d] . Q^T[d][head]      (16 tokens on M; A fragments by ldmatrix)
//   O^T[d][head]   += V^T[d][token] . P[token][head]  (16 dims per tile; A fragments by ldmatrix.trans)
// A lane holds the logits of two heads for two tokens; the probabilities become the B operand of
// the second product through one movmatrix transpose per 8-token half. bf16 products are exact in
// fp32; P is split into a bf16 high part and a bf16 remainder (two MMAs) so that the weighted sum
// keeps about 16 bits of P. The online softmax keeps per-head running maxima that are raised only
// when a logit exceeds them by more than 2^8, so the rescale branch is rare.
#include "kernels.h"

#include <cooperative_groups.h>
#include <cuda_bf16.h>


namespace cg = cooperative_groups;

namespace fastocr {
namespace {

constexpr int kStages = 3;
constexpr int kThreads = kAttnWarps * 32;
constexpr int kBlockTokens = 16;                        // tokens per warp per pipeline stage
constexpr int kRowTokens = kAttnWarps * kBlockTokens;   // tokens per CTA per pipeline stage
constexpr float kRescaleSlack = 8.0f;                   // log2 units
constexpr int kMergePitch = kHeadDim + 4;                // floats per head in the CTA's merge buffer (bank spread)
constexpr int kMergeRound = 4;                          // partials fetched together by the merging CTA
constexpr int kLongRangeRows = 128;                     // rows per CTA from which unit alignment is dropped

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Cache rows are read once per layer: they go through L2 marked evict-first, so that streaming a
// gigabyte of them does not push out what is read again soon (the logits of a focal layer, the
// index list, the queries).
__device__ __forceinline__ uint64_t l2_evict_first_policy() { return l2_policy_evict_first(); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// four 8x8 b16 matrices from shared memory (lane l supplies the address of row l % 8 of matrix l / 8)
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// transpose of an 8x8 b16 matrix held one row per lane group (the MMA fragment layout)
__device__ __forceinline__ uint32_t movm_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// two adjacent outputs (even index), bf16 or fp32
__device__ __forceinline__ void store_pair(void* out, int is_fp32, int64_t index, float x, float y) {
  if (is_fp32) *reinterpret_cast<float2*>(reinterpret_cast<float*>(out) + index) = make_float2(x, y);
  else *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(out) + index) = __floats2bfloat162_rn(x, y);
}

// number of attended tokens of sequence b and the pieces needed to enumerate them
struct SeqGeom {
  int vs, N, kept_vis, n_tok;                           // n_tok: attended tokens of this launch (< 0: the sequence takes no part)
};
// The lengths come from device memory and cannot be checked by the host without a synchronisation:
// they are forced into what the host did check (0 <= seq_len <= max_seq_len, the image span inside
// the sequence, the kept count inside the span and inside the index list's row), so that no cache
// row, block-table entry or index-list entry outside the caller's buffers is ever addressed. `bad`
// counts the lengths that had to be changed (a kept count above the span or the row length is
// documented behaviour, not a fault).
__device__ __forceinline__ SeqGeom load_geom(const AttnLaunch& a, int b, bool pruned, int& bad) {
  SeqGeom s;
  const int S_in = a.seq_len[b], vs_in = a.vis_start[b], N_in = a.vis_len[b];
  const int S = min(max(S_in, 0), a.max_seq_len);
  s.vs = min(max(vs_in, 0), S);
  s.N = min(max(N_in, 0), S - s.vs);
  bad += (S != S_in) + (s.vs != vs_in) + (s.N != N_in);
  if (pruned) {
    const int kk = a.kcount[b];
    s.kept_vis = min(max(kk, 0), min(s.N, a.k_stride));
  } else {
    s.kept_vis = s.N;
  }
  s.n_tok = S - s.N + s.kept_vis;
  if (a.seq_mask != nullptr && a.seq_mask[b] != a.mask_want) s.n_tok = -1;
  return s;
}
__device__ __forceinline__ SeqGeom load_geom(const AttnLaunch& a, int b, bool pruned) {
  int ignored = 0;
  return load_geom(a, b, pruned, ignored);
}

// chunk swizzle of a staged row (16 chunks of 16 bytes): the eight rows of an ldmatrix 8x8 matrix
// (eight consecutive tokens, same chunk) land in eight different 16-byte bank groups
__device__ __forceinline__ int row_swz(int tok) { return tok & 7; }

// shared-memory carve-up (bytes). A stage holds a 16 x 256 B K tile (+ the same for V) per warp.
template <bool HAS_V>
struct Smem {
  static constexpr int kTileBytes = kBlockTokens * kHeadDim * 2;
  static constexpr int kStageBytes = (HAS_V ? 2 : 1) * kTileBytes;   // per warp
  static constexpr int kRingBytes = kAttnWarps * kStages * kStageBytes;
  static constexpr int ring = 0;
  static constexpr int prefix = kRingBytes;                          // int32 [kMaxUnits + 1], rows before each unit
  static constexpr int merge = prefix + ((kMaxUnits + 1) * 4 + 15) / 16 * 16;   // float m[8], l[8], o[8][128], int flag
  static constexpr int total = merge + (16 + kMaxGroup * (kHeadDim + 4) + 4) * 4;
};

#ifdef FASTOCR_TRACE
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define FASTOCR_TRACE_CLK(var) const long long var = clock64()
#define FASTOCR_TRACE_CYC(slot)                                                                             \
  do {                                                                                                      \
    if (a.trace != nullptr && lane == 0) a.trace[(blockIdx.x * kAttnWarps + warp) * 16 + (slot)] = clock64(); \
  } while (0)
#define FASTOCR_TRACE_ADD(acc, t1, t0) acc += static_cast<unsigned>((t1) - (t0))
#define FASTOCR_TRACE_MARK(slot)                                                                            \
  do {                                                                                                      \
    if (a.trace != nullptr && lane == 0) a.trace[(blockIdx.x * kAttnWarps + warp) * 16 + (slot)] = trace_now(); \
  } while (0)
#else
#define FASTOCR_TRACE_MARK(slot) do { } while (0)
#define FASTOCR_TRACE_CLK(var) do { } while (0)
#define FASTOCR_TRACE_CYC(slot) do { } while (0)
#define FASTOCR_TRACE_ADD(acc, t1, t0) do { } while (0)
#endif

// Ways to hand out rows (see the kernel): 0 = equal ranges of all rows laid end to end; else every
// unit is cut into this many equal parts, one CTA each. Units of similar length get as many parts as
// the grid allows. A ragged batch of index-list units gets one CTA per unit when the units number at
// least a fifth of the grid and none is far longer than the average: the CTAs then finish at
// different times, but none shares a unit with another, so there are no partial results through
// global memory, hence no waiting for the previous kernel, and the next layers' launches (two or
// three are in flight) fill the idle slots. (Full-cache passes overlap far less and their units are
// long: one CTA per unit left them 2.6x slower than equal ranges, so they keep the ranges.)
constexpr int kOwnUnitMaxRows = 512;
__device__ __forceinline__ int split_rule(int units, int grid, int total_rows, int longest_unit, bool index_list) {
  if (units > grid || total_rows >= kLongRangeRows * grid) return 0;
  const int64_t padded = static_cast<int64_t>(longest_unit) * units;
  if (padded <= static_cast<int64_t>(total_rows) + total_rows / 8) return min(grid / units, kMaxPartsPerUnit);
  return (index_list && 5 * units >= grid && longest_unit <= kOwnUnitMaxRows && padded <= 2 * static_cast<int64_t>(total_rows)) ? 1 : 0;
}

// A unit cut into `parts` pieces whose CTAs were launched as one thread-block cluster of that size
// (CTA index / parts = unit, so cluster = unit) is merged inside the cluster. The answer is the same
// in every CTA of a cluster: all derive the split from the same lengths and the same grid.
__device__ __forceinline__ bool merges_in_cluster(bool split_units, int parts) {
  return split_units && parts > 1 && static_cast<int>(cg::this_cluster().num_blocks()) == parts;
}

// What a launch does is fixed at compile time, so that the main loop carries no code it does not
// run (the page-table arithmetic alone, present but skipped, cost a pruned pass 6 %):
//   kModePruned  K = T u F: index list, K and V, no logits   (copy distance 3: more latency hidden per warp)
//   kModeScores  full cache, K and V, logits and per-head statistics kept for the selection
//   kModeDense   full cache, K and V
//   kModeKeys    full cache, K only, logits and statistics (stand-alone scoring)
// (copy distance 2 for the full-cache passes: they saturate HBM anyway and run faster with fewer
// requests queued), each for contiguous and for paged caches.
enum : int { kModePruned = 0, kModeScores = 1, kModeDense = 2, kModeKeys = 3 };

template <int G, int MODE, bool PAGED>
__global__ void __launch_bounds__(kThreads, kAttnCtasPerSm) attn_stream_kernel(const AttnLaunch a) {
  constexpr bool HAS_V = MODE != kModeKeys;
  constexpr bool HAS_IDX = MODE == kModePruned;
  constexpr bool LOGITS = MODE == kModeScores || MODE == kModeKeys;
  constexpr int kDepth = MODE == kModePruned ? 3 : 2;   // blocks a copy is issued ahead of its use (<= kStages)
  static_assert(kDepth >= 1 && kDepth <= kStages, "copy distance");
  extern __shared__ __align__(16) unsigned char smem[];
  using L = Smem<HAS_V>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g8 = lane >> 2, t4 = lane & 3;             // MMA fragment coordinates: group, thread-in-group
  const int Hkv = a.num_kv_heads;
  const int units = a.batch * Hkv;                     // unit u = (sequence u / Hkv, KV head u % Hkv)

  FASTOCR_TRACE_MARK(0);
  FASTOCR_TRACE_CYC(8);
#ifdef FASTOCR_TRACE
  unsigned trace_wait = 0, trace_qk = 0, trace_look = 0, trace_pv = 0;   // cycles, summed over the main loop
#endif
  // Everything read before the first wait_for_prior_grids() must not have been produced by a
  // kernel that may still be running; the host says how much that is (AttnLaunch::wait_point).
  // The next kernel is let in only once this one's own early reads are known to be safe: a kernel
  // whose inputs were settled before it started says so at once, the others after their wait
  // (their successor may assume that whatever they waited for has completed).
  if (a.wait_point == kWaitAtStart) wait_for_prior_grids();
  if (a.wait_point != kWaitAfterSetup) dependents_may_launch();

  // ---- set-up: prefix of the units' row counts ----------------------------------------------------
  // Every thread fetches the lengths of up to kMaxUnits / kThreads units at once (one round trip to
  // L2 for the whole table), warp 0 then scans the counts in shared memory.
  int* prefix_s = reinterpret_cast<int*>(smem + L::prefix);
  float* mrg_m = reinterpret_cast<float*>(smem + L::merge);   // [8]
  float* mrg_l = mrg_m + 8;                                    // [8]
  float* mrg_o = mrg_m + 16;                                   // [8][kMergePitch]
  int* mrg_flag = reinterpret_cast<int*>(mrg_o + kMaxGroup * kMergePitch);
  // every unit's geometry, kept in the (still unused) ring until the CTA has picked up that of its
  // first unit: saves that unit a second round trip to L2
  int4* geom_s = reinterpret_cast<int4*>(smem + L::ring);
  static_assert(kMaxUnits * 16 <= L::kRingBytes, "the geometry table must fit the ring");
  // A launch plan (launch_attn_plan) hands the CTA its range, its unit and the unit's geometry
  // in one 64-byte record: one round trip and no scan. A record marked invalid (the CTA's range
  // would span several units) sends the CTA through the full set-up.
  if (tid == 0) mrg_flag[3] = 0;
  __syncthreads();
  int bad_lengths = 0;                                 // CTA 0: device-side lengths outside what the host checked
  int4 plan0 = make_int4(0, 0, 0, 0), plan1 = plan0, plan2 = plan0, plan3 = plan0;
  if (a.plan != nullptr) {
    const int4* rec = a.plan + 4 * static_cast<int64_t>(blockIdx.x);
    plan0 = __ldg(rec);
    plan1 = __ldg(rec + 1);
    plan2 = __ldg(rec + 2);
    plan3 = __ldg(rec + 3);
  }
  const bool planned = plan0.x != 0;
  //                  // {valid, unit, r0, r1} {ubeg, uend, split, parts} {per_cta, total, -, -} {geometry}
  if (planned) {
    if (tid == 0) {
      prefix_s[plan0.y] = plan1.x;
      prefix_s[plan0.y + 1] = plan1.y;
      prefix_s[units] = plan2.y;
      geom_s[plan0.y] = plan3;
    }
  } else {
    constexpr int kPerThread = kMaxUnits / kThreads;
    SeqGeom gq[kPerThread];                            // all loads first, so that they are in flight together
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int uu = min(i * kThreads + tid, units - 1);
      int bad = 0;
      gq[i] = load_geom(a, uu / Hkv, HAS_IDX, bad);
      // lengths that had to be forced into range: counted once per launch and sequence
      if (blockIdx.x == 0 && i * kThreads + tid < units && uu % Hkv == 0) bad_lengths += bad;
    }
    int longest = 0;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int uu = i * kThreads + tid;
      if (uu < units) {
        const int rows = (gq[i].n_tok + kRowTokens - 1) / kRowTokens;
        geom_s[uu] = make_int4(gq[i].vs, gq[i].N, gq[i].kept_vis, gq[i].n_tok);
        prefix_s[uu + 1] = rows;
        longest = max(longest, rows);
        if (gq[i].n_tok == 0) mrg_flag[3] = 1;         // some unit has nothing to attend (rare)
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) longest = max(longest, __shfl_xor_sync(0xffffffffu, longest, o));
    if (lane == 0) mrg_flag[1 + warp] = longest;
  }
  FASTOCR_TRACE_CYC(9);
  __syncthreads();
  if (warp == 0 && !planned) {                         // lane l owns units [l * chunk, (l + 1) * chunk)
    const int chunk = (units + 31) >> 5;
    const int u_lo = lane * chunk, u_hi = min(units, u_lo + chunk);
    int sum = 0;
    for (int uu = u_lo; uu < u_hi; ++uu) sum += prefix_s[uu + 1];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    int run = incl - sum;
    for (int uu = u_lo; uu < u_hi; ++uu) {
      run += prefix_s[uu + 1];
      prefix_s[uu + 1] = run;
    }
    if (lane == 0) {
      prefix_s[0] = 0;
      int longest = mrg_flag[1];
#pragma unroll
      for (int w = 1; w < kAttnWarps; ++w) longest = max(longest, mrg_flag[1 + w]);
      mrg_flag[1] = longest;
    }
  }
  __syncthreads();
  FASTOCR_TRACE_MARK(1);
  FASTOCR_TRACE_CYC(10);
  const int total_rows = prefix_s[units], longest_unit = planned ? 0 : mrg_flag[1];
  const int grid = min(static_cast<int>(gridDim.x), a.active_ctas);
  // Two ways to hand out rows. Short ranges over at most `grid` units of similar length: every unit
  // is cut into the same number of equal parts, one per CTA, so no CTA straddles two units (no
  // pipeline refill) and a unit that fits one CTA needs no global merge. Otherwise (ragged
  // batches, more units than CTAs, or long ranges where a few merges are negligible): all rows
  // laid end to end and cut into equal ranges.
  // A group of layers (pruned passes only): the rows of all its layers, layer after layer, are one long
  // sequence cut into equal ranges. A CTA streams through its range without regard to unit or layer
  // boundaries; the few units it shares with its neighbours are merged through global partials.
  const int n_layers = HAS_IDX ? max(a.n_layers, 1) : 1;
  const bool grouped = n_layers > 1;
  const int all_rows = n_layers * total_rows;          // rows of the launch
  const int parts_rule = (planned || grouped) ? 0 : split_rule(units, grid, total_rows, longest_unit, HAS_IDX);
  const bool split_units = planned ? plan1.z != 0 : parts_rule > 0;
  const int parts = planned ? plan1.w : max(parts_rule, 1);     // CTAs per unit
  const int per_cta = planned ? plan2.x : (all_rows + grid - 1) / grid;   // rows per CTA (equal-range mode)
  int r0 = 0, r1 = 0, first_unit = 0;
  if (planned) {
    first_unit = plan0.y;
    r0 = plan0.z;
    r1 = plan0.w;
  } else if (static_cast<int>(blockIdx.x) >= grid) {
    // a spare CTA: launched only so that the launch claims the whole shared-memory array of every SM
  } else if (split_units) {
    first_unit = blockIdx.x / parts;
    if (first_unit < units) {
      const int ub = prefix_s[first_unit], ue = prefix_s[first_unit + 1];
      const int per = (ue - ub + parts - 1) / parts;
      r0 = min(ue, ub + (blockIdx.x - first_unit * parts) * per);
      r1 = min(ue, r0 + per);
    }
  } else {
    r0 = min(all_rows, static_cast<int>(blockIdx.x) * per_cta);
    r1 = min(all_rows, r0 + per_cta);
  }

  const float scale_log2 = a.sm_scale * 1.4426950408889634f;
  const int64_t row_elems = static_cast<int64_t>(Hkv) * kHeadDim;
  const int64_t seq_elems = PAGED ? 0 : a.seq_stride_tokens * row_elems;
  const int c16 = lane & 15, half = lane >> 4;          // copy role: chunk of a row, which row of a pair
  const uint32_t smem_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const uint32_t ring_warp = smem_u32 + L::ring + warp * kStages * L::kStageBytes;
  const bool head_ok = g8 < G;
  const int row_bytes = Hkv * kHeadDim * 2;
  // ldmatrix row addresses inside a tile (lane l gives row l % 8 of matrix i = l / 8). K (A operand
  // of S = K Q^T, tokens on M): matrix i = (tokens 8 (i & 1) .., chunk 2 s + (i >> 1)); V (A operand
  // of O^T = V^T P through .trans): matrix i = (tokens 8 (i >> 1) .., chunk 2 j + (i & 1)). Steps s
  // and s + 4 differ by 8 chunks = 128 bytes, which the swizzle (bits 0-2 of the chunk) leaves alone.
  uint32_t k_off[4], v_off[4];
  {
    const int lm_r = lane & 7, lm_i = lane >> 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      k_off[i] = (lm_r + 8 * (lm_i & 1)) * 256 + (((2 * i + (lm_i >> 1)) ^ lm_r) << 4);
      v_off[i] = (lm_r + 8 * (lm_i >> 1)) * 256 + (((2 * i + (lm_i & 1)) ^ lm_r) << 4);
    }
  }
  // where this lane's 16-byte chunk of rows 2i + half of a tile lands (rows 2i + 8 + half: 2048 bytes further)
  uint32_t cp_off[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) cp_off[i] = (2 * i + half) * 256 + ((c16 ^ row_swz(2 * i + half)) << 4);
  const uint64_t stream_policy = l2_evict_first_policy();
  const uint64_t keep_policy = LOGITS ? l2_policy_evict_last() : 0;   // logits: read back by the next kernel

  // ---- the CTA's range, one unit segment after the other --------------------------------------
  int u = first_unit;
  int layer = 0, layer_row0 = 0;                       // layer of the group the walk is in, and its first row
  if (!planned && !split_units && r0 < r1) {
    if (grouped) {
      layer = r0 / total_rows;
      layer_row0 = layer * total_rows;
    }
    const int local = r0 - layer_row0;
    int lo = 0, hi = units;                            // largest u with prefix[u] <= local
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (prefix_s[mid] <= local) lo = mid; else hi = mid;
    }
    u = lo;
  }
  int seg_begin = r0;
  int bad_entries = 0;                                 // index-list entries outside the image span (clamped), counted by lanes 0-15
  if (a.wait_point == kWaitAfterSetup) {               // before index-list reads and logits writes
    wait_for_prior_grids();
    dependents_may_launch();
  }
  FASTOCR_TRACE_MARK(2);                               // (debug builds) the wait, if any, is over
  // State that survives a segment boundary when the look-ahead stages of one segment have already
  // fetched the first blocks of the next (see `carry_next` below).
  uint32_t qb[8][2];                                   // B fragments of Q^T of the segment's unit
  bool carried = false;                                // this segment's first blocks are in flight already, q is loaded
  int pos_p = 0, row_p = 0;
  bool idx_p = false;
  const uint32_t ring_end = ring_warp + kStages * L::kStageBytes;
  uint32_t src = ring_warp, dst_ahead = ring_warp;     // ring slots of block n and of block n + kDepth
#pragma unroll 1
  while (seg_begin < r1) {
    while (true) {                                     // skip empty units; past the last unit the next layer begins
      if (grouped && u == units) {
        u = 0;
        ++layer;
        layer_row0 += total_rows;
      }
      if (layer_row0 + prefix_s[u + 1] > seg_begin) break;
      ++u;
    }
    const int ubeg = layer_row0 + prefix_s[u], uend = layer_row0 + prefix_s[u + 1];
    const int seg_rows = min(uend, r1) - seg_begin;    // rows of unit u inside this range
    const int b = u / Hkv, g = u - b * Hkv;
    SeqGeom sg;
    if (seg_begin == r0) {                             // first segment: from the table in shared memory
      const int4 gq = geom_s[u];
      sg.vs = gq.x; sg.N = gq.y; sg.kept_vis = gq.z; sg.n_tok = gq.w;
      __syncthreads();                                 // both warps have read it: the ring may be written
    } else {
      sg = load_geom(a, b, HAS_IDX);
    }
    const int tok0 = (seg_begin - ubeg) * kRowTokens + warp * kBlockTokens;   // this warp's first token of the segment
    // this lane's 16-byte chunk of cache row 0 of the unit (a row is row_bytes long)
    const void* k_base = grouped ? a.layer_k[layer] : a.k;
    const void* v_base = grouped ? a.layer_v[layer] : a.v;
    const char* kptr = reinterpret_cast<const char*>(k_base) + (b * seq_elems + g * kHeadDim + 8 * c16) * 2;
    const char* vptr = HAS_V ? reinterpret_cast<const char*>(v_base) + (b * seq_elems + g * kHeadDim + 8 * c16) * 2 : nullptr;

    // B fragments of Q^T for the eight 16-dim steps: head g8, dims 16 s + {2 t4, 2 t4 + 1} and 16 s + 8 + {2 t4, 2 t4 + 1}
    auto load_q = [&](int unit) {
      const uint32_t* qp = reinterpret_cast<const uint32_t*>(static_cast<const char*>(a.q) + layer * a.q_layer_bytes) +
                           (static_cast<int64_t>(unit) * G + g8) * (kHeadDim / 2) + t4;
#pragma unroll
      for (int st = 0; st < 8; ++st) {
        qb[st][0] = head_ok ? __ldg(qp + 8 * st) : 0u;
        qb[st][1] = head_ok ? __ldg(qp + 8 * st + 4) : 0u;
      }
    };
    if (!carried) load_q(u);
    // The lane's share of the state: heads hA = 2 t4 and hB = 2 t4 + 1.
    float o[8][4];                                     // O^T tile j: dims {16 j + g8, 16 j + 8 + g8} x heads {hA, hB}
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
    float mA = -INFINITY, mB = -INFINITY;              // reference maxima (identical in the 8 lanes that share t4)
    float lA = 0.f, lB = 0.f;                          // this lane's part of the sums (tokens g8, 8 + g8 of every block)
    const bool okA = 2 * t4 < G, okB = 2 * t4 + 1 < G;
    float* logitA = (LOGITS && okA) ? a.logits + (static_cast<int64_t>(u) * G + 2 * t4) * a.n_stride : nullptr;
    float* logitB = (LOGITS && okB) ? a.logits + (static_cast<int64_t>(u) * G + 2 * t4 + 1) * a.n_stride : nullptr;

    // Look-ahead stages, each one block behind the previous (so that no loaded value is needed in
    // the iteration that loads it): P (block n + kDepth + 2) logical position of token `lane % 16`
    // of this warp's block, a load from the index list for selected image tokens; R (block
    // n + kDepth + 1) physical cache row, a block-table load for paged caches; I (block n + kDepth)
    // the cp.async copies; C (block n) the arithmetic.
    // A block is named by the list index jr of its first token (tok0 + 32 per block); it exists
    // while jr < lim. All 32 lanes run stages P and R (lanes 16-31 mirror lanes 0-15: no divergence).
    const int lim = min(sg.n_tok, tok0 + seg_rows * kRowTokens);
    // When the range goes on into the next KV head of the same sequence (same lengths, same index
    // list, same block table; the cache rows lie 256 bytes further), the look-ahead stages do not idle
    // over the last blocks of this segment: they fetch the first blocks of the next one, which then
    // starts with its pipeline full, no prologue, no drain in between. (Other boundaries: next
    // sequence, next layer, a short segment: the pipeline is drained and refilled.)
    const int seg_tok_end = tok0 + seg_rows * kRowTokens;          // list index at which this warp leaves the segment
    bool carry_next = false;
    int lim_n = 0;                                                 // the next segment's limit; 0: nothing to fetch there
    if (!planned && !split_units && seg_begin + seg_rows < r1 && seg_rows >= kDepth + 2 && u + 1 < units && (u + 1) / Hkv == b) {
      const int rows_n = min(layer_row0 + prefix_s[u + 2], r1) - (seg_begin + seg_rows);
      if (prefix_s[u + 2] > prefix_s[u + 1] && rows_n > 0) {
        carry_next = true;
        lim_n = min(sg.n_tok, warp * kBlockTokens + rows_n * kRowTokens);
      }
    }
    const int shift_n = seg_tok_end - warp * kBlockTokens;         // list index in this segment -> list index in the next
    const int tl = lane & (kBlockTokens - 1);
    const int vis_end = sg.vs + sg.kept_vis, text_shift = sg.N - sg.kept_vis;
    const int32_t* idx_row = HAS_IDX ? a.idx + static_cast<int64_t>(b) * a.k_stride - sg.vs : nullptr;
    const int32_t* bt_row = PAGED ? a.block_table + static_cast<int64_t>(b) * a.max_pages : nullptr;
    // A look-ahead block named by a list index past the end of this segment belongs to the next one.
    auto locate = [&](int& jr, int& lx, int& head_off) {
      lx = lim;
      head_off = 0;
      if (jr >= seg_tok_end) {
        jr -= shift_n;
        lx = lim_n;
        head_off = kHeadDim * 2;
      }
    };
    auto stage_p = [&](int jr, int lx, int& pos, bool& is_idx) {     // is_idx: pos is a raw index-list entry, checked in stage R
      is_idx = false;
      if (jr < lx) {
        const int j = min(jr + tl, sg.n_tok - 1);
        pos = j;
        if (HAS_IDX) {                                 // kept set: text before | selected image | text after
          if (j >= vis_end) {
            pos = j + text_shift;
          } else if (j >= sg.vs) {
            pos = __ldg(idx_row + j);
            is_idx = true;
          }
        }
      }
    };
    auto stage_r = [&](int jr, int lx, int pos, bool is_idx, int& row) {
      if (jr < lx) {
        if (is_idx) {
          const int inside = min(max(pos, 0), sg.N - 1);      // never read outside the image span
          bad_entries += inside != pos;
          pos = inside + sg.vs;
        }
        if (PAGED) {
          int page = __ldg(bt_row + (pos >> a.page_shift));         // page sizes are powers of two
          if (a.num_pages > 0) {                                    // never read outside the pool
            const int inside = min(max(page, 0), a.num_pages - 1);
            bad_entries += inside != page;
            page = inside;
          }
          pos = (page << a.page_shift) + (pos & (a.page_size - 1));
        }
        row = pos;
      }
    };
    // The copies of a block: its 16 K rows are one cp.async group, its 16 V rows another (K is
    // needed at the top of the block's iteration, V only after the softmax, and each tile's ring
    // slot is free again as soon as the fragments of the block that used it last are in registers).
    auto stage_ik = [&](int jr, int lx, int head_off, uint32_t dst, int row) {
      if (jr < lx) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {                  // rows 2i (lanes 0-15) and 2i + 1 (lanes 16-31)
          const int rr = __shfl_sync(0xffffffffu, row, 2 * i + half);
          cp_async16(dst + cp_off[i & 3] + (i >> 2) * 2048, kptr + head_off + static_cast<int64_t>(rr) * row_bytes, stream_policy);
        }
      }
      cp_async_commit();
    };
    auto stage_iv = [&](int jr, int lx, int head_off, uint32_t dst, int row) {
      if (!HAS_V) return;
      if (jr < lx) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rr = __shfl_sync(0xffffffffu, row, 2 * i + half);
          cp_async16(dst + L::kTileBytes + cp_off[i & 3] + (i >> 2) * 2048, vptr + head_off + static_cast<int64_t>(rr) * row_bytes, stream_policy);
        }
      }
      cp_async_commit();
    };
    // groups younger than the one waited for: K(n) at the top of iteration n, V(n) before P.V
    constexpr int kWaitK = HAS_V ? 2 * kDepth - 1 : kDepth - 1;
    constexpr int kWaitV = 2 * kDepth - 1;
    // Address translation: a pruned pass touches a handful of rows in every 2 MiB page of the
    // sequence's cache span, and the first touch of a page by this SM costs a translation miss in
    // the middle of the stream. Touch every page of the span now, all at once (one line each, L2
    // only): lanes 0-15 of warp 0 for K, lanes 16-31 for V.
    if (HAS_IDX && !PAGED && warp == 0 && !carried) {
      const int64_t span = static_cast<int64_t>(sg.n_tok - sg.kept_vis + sg.N) * row_elems * 2;   // bytes, whole sequence
      const char* base = reinterpret_cast<const char*>(half ? v_base : k_base) + (b * seq_elems + g * kHeadDim) * 2;
      int64_t off = static_cast<int64_t>(c16) << 21;
      if (c16 == 15) off = span - 256;
      if (off >= 0 && off < span && (HAS_V || half == 0)) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
    }
    // Filling the stages: the lookups of the first rows are issued together (one round trip for
    // the index-list entries, one for the block-table entries) instead of one after the other,
    // then the copies of the first kDepth rows go out.
    FASTOCR_TRACE_CYC(11);
    if (!carried) {
      // (a segment shorter than the look-ahead names blocks past its end here: they are looked for in
      // the next segment only by the main loop, so they must not exist for the prologue)
      int posq[kDepth + 2], rowq[kDepth + 1];
      bool ixq[kDepth + 2];
#pragma unroll
      for (int r = 0; r < kDepth + 2; ++r) {
        posq[r] = 0;
        stage_p(tok0 + r * kRowTokens, lim, posq[r], ixq[r]);
      }
#pragma unroll
      for (int r = 0; r < kDepth + 1; ++r) {
        rowq[r] = 0;
        stage_r(tok0 + r * kRowTokens, lim, posq[r], ixq[r], rowq[r]);
      }
      FASTOCR_TRACE_CYC(12);
#pragma unroll
      for (int r = 0; r < kDepth; ++r) {
        stage_ik(tok0 + r * kRowTokens, lim, 0, ring_warp + (r % kStages) * L::kStageBytes, rowq[r]);
        stage_iv(tok0 + r * kRowTokens, lim, 0, ring_warp + (r % kStages) * L::kStageBytes, rowq[r]);
      }
      row_p = rowq[kDepth];
      pos_p = posq[kDepth + 1];
      idx_p = ixq[kDepth + 1];
      src = ring_warp;
      dst_ahead = ring_warp + (kDepth % kStages) * L::kStageBytes;
      FASTOCR_TRACE_CYC(13);
    }
#pragma unroll 1
    for (int j0 = tok0; j0 < tok0 + seg_rows * kRowTokens; j0 += kRowTokens) {   // j0: list index of the block's first token
      FASTOCR_TRACE_CLK(c_top);
      cp_async_wait<kWaitK>();
      __syncwarp();                                    // every lane's K copies of this block have landed
      FASTOCR_TRACE_CLK(c_waited);
      FASTOCR_TRACE_ADD(trace_wait, c_waited, c_top);
      if (j0 == tok0 && seg_begin == r0) { FASTOCR_TRACE_MARK(3); FASTOCR_TRACE_CYC(14); }   // first data of the CTA's range
      const bool live = j0 < sg.n_tok;                 // the block holds at least one attended token
      // two accumulators (even / odd 16-dim steps): dependent MMA chains of four
      float sc[4] = {0.f, 0.f, 0.f, 0.f}, sc2[4] = {0.f, 0.f, 0.f, 0.f};
      if (live) {
        // ---- S = K Q^T: tokens j0 + {g8, 8 + g8} x heads {hA, hB} ---------------------------------
#pragma unroll
        for (int st = 0; st < 8; ++st) {
          uint32_t ka[4];
          ldsm_x4(ka, src + k_off[st & 3] + (st >> 2) * 128);
          if (st & 1) mma_bf16(sc2, ka[0], ka[1], ka[2], ka[3], qb[st][0], qb[st][1]);
          else mma_bf16(sc, ka[0], ka[1], ka[2], ka[3], qb[st][0], qb[st][1]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[i] += sc2[i];
      }
      FASTOCR_TRACE_CLK(c_qk);
      FASTOCR_TRACE_ADD(trace_qk, c_qk, c_waited);
      // ---- look-ahead: K copies of block n + kDepth into the slot block n's K tile just left, then
      // stages R and P one and two blocks further ---------------------------------------------------
      __syncwarp();                                    // every lane has this block's K fragments
      int jr_i = j0 + kDepth * kRowTokens, lim_i, off_i;
      locate(jr_i, lim_i, off_i);
      stage_ik(jr_i, lim_i, off_i, dst_ahead, row_p);
      const int row_v = row_p;
      {
        int jr = j0 + (kDepth + 1) * kRowTokens, lx, off;
        locate(jr, lx, off);
        stage_r(jr, lx, pos_p, idx_p, row_p);
        jr = j0 + (kDepth + 2) * kRowTokens;
        locate(jr, lx, off);
        stage_p(jr, lx, pos_p, idx_p);
      }

      FASTOCR_TRACE_CLK(c_look);
      FASTOCR_TRACE_ADD(trace_look, c_look, c_qk);
      if (live) {
        // ---- online softmax: x[0], x[1] token j0 + g8 (heads hA, hB); x[2], x[3] token j0 + 8 + g8 ------
        float x[4] = {sc[0] * scale_log2, sc[1] * scale_log2, sc[2] * scale_log2, sc[3] * scale_log2};
        const int rem = sg.n_tok - j0 - g8;            // > 0: token j0 + g8 is attended; > 8: token j0 + 8 + g8 too
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int tok = j0 + g8 + 8 * (i >> 1);      // index in the unit's attended list
          const bool valid = ((i & 1) ? okB : okA) && rem > 8 * (i >> 1);
          x[i] = valid ? x[i] : -INFINITY;
          float* lrow = (i & 1) ? logitB : logitA;
          if (LOGITS && lrow != nullptr && valid) {              // dense / scoring mode: position == list index
            const int rel = tok - sg.vs;
            if (rel >= 0 && rel < sg.N && rel < a.n_stride) store_logit(lrow + rel, x[i], keep_policy);
          }
        }
        float mxA = fmaxf(x[0], x[2]), mxB = fmaxf(x[1], x[3]);
        if (__builtin_expect(__any_sync(0xffffffffu, mxA > mA + kRescaleSlack || mxB > mB + kRescaleSlack), 0)) {
#pragma unroll
          for (int off = 4; off < 32; off <<= 1) {     // over the 8 lanes that share t4
            mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, off));
            mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, off));
          }
          const bool raiseA = mxA > mA + kRescaleSlack, raiseB = mxB > mB + kRescaleSlack;
          const float alA = raiseA ? fast_exp2(mA - mxA) : 1.f;   // m = -inf gives 0
          const float alB = raiseB ? fast_exp2(mB - mxB) : 1.f;
          if (raiseA) mA = mxA;
          if (raiseB) mB = mxB;
          lA *= alA;
          lB *= alB;
          if (HAS_V) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              o[j][0] *= alA; o[j][1] *= alB; o[j][2] *= alA; o[j][3] *= alB;
            }
          }
        }
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = (x[i] == -INFINITY) ? 0.f : fast_exp2(x[i] - ((i & 1) ? mB : mA));
        lA += p[0] + p[2];
        lB += p[1] + p[3];
        if (HAS_V) {
          // P as the B operand of O^T += V^T P (tokens on K, head g8 on N) is the transpose of what the
          // lanes hold (token g8, heads hA hB): one movmatrix per 8-token half, for the bf16 high
          // part and for the remainder
          const uint32_t h0 = pack_bf16(p[0], p[1]), h1 = pack_bf16(p[2], p[3]);
          const uint32_t r0w = pack_bf16(p[0] - __uint_as_float(h0 << 16), p[1] - __uint_as_float(h0 & 0xffff0000u));
          const uint32_t r1w = pack_bf16(p[2] - __uint_as_float(h1 << 16), p[3] - __uint_as_float(h1 & 0xffff0000u));
          const uint32_t ph0 = movm_trans(h0), ph1 = movm_trans(h1), pl0 = movm_trans(r0w), pl1 = movm_trans(r1w);
          cp_async_wait<kWaitV>();
          __syncwarp();                                // every lane's V copies of this block have landed
          uint32_t va[8][4];                           // A fragments of V^T: dims 16 j .. + 15 x the block's 16 tokens
#pragma unroll
          for (int j = 0; j < 8; ++j) ldsm_x4_trans(va[j], src + L::kTileBytes + v_off[j & 3] + (j >> 2) * 128);
          __syncwarp();                                // the V tile's slot is free: copies of block n + kDepth
          stage_iv(jr_i, lim_i, off_i, dst_ahead, row_v);         // go out while the tensor cores work
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mma_bf16(o[j], va[j][0], va[j][1], va[j][2], va[j][3], ph0, ph1);
            mma_bf16(o[j], va[j][0], va[j][1], va[j][2], va[j][3], pl0, pl1);
          }
        }
      }
      if (HAS_V && !live) stage_iv(jr_i, lim_i, off_i, dst_ahead, row_v);   // keeps the group count in step
      src += L::kStageBytes;
      if (src == ring_end) src = ring_warp;
      dst_ahead += L::kStageBytes;
      if (dst_ahead == ring_end) dst_ahead = ring_warp;
      FASTOCR_TRACE_CLK(c_end);
      FASTOCR_TRACE_ADD(trace_pv, c_end, c_look);
    }
    if (carry_next) load_q(u + 1);                     // the next segment's queries arrive while this one is merged
    else cp_async_wait<0>();
    FASTOCR_TRACE_MARK(4);
    FASTOCR_TRACE_CYC(15);

    // ---- leaving the unit (all warps of the CTA get here together: they walk the same rows) ----------
    // sums over the block's tokens: the 8 lanes that share t4 hold parts for heads hA, hB
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      lA += __shfl_xor_sync(0xffffffffu, lA, off);
      lB += __shfl_xor_sync(0xffffffffu, lB, off);
    }
    __syncthreads();                                   // the merge buffer is free again
    // the warps fold their state into the shared buffer, one after the other
#pragma unroll 1
    for (int w = 0; w < kAttnWarps; ++w) {
      if (warp == w) {
        float sbA = 0.f, swA = 1.f, sbB = 0.f, swB = 1.f, MnA = mA, MnB = mB;
        if (w > 0) {
          const float bA = mrg_m[2 * t4], bB = mrg_m[2 * t4 + 1];
          MnA = fmaxf(bA, mA);
          MnB = fmaxf(bB, mB);
          sbA = bA == -INFINITY ? 0.f : exp2f(bA - MnA); swA = mA == -INFINITY ? 0.f : exp2f(mA - MnA);
          sbB = bB == -INFINITY ? 0.f : exp2f(bB - MnB); swB = mB == -INFINITY ? 0.f : exp2f(mB - MnB);
        }
        __syncwarp();                                  // every lane has read the old maxima
        if (g8 == 0) {
          mrg_l[2 * t4] = (w > 0 ? mrg_l[2 * t4] * sbA : 0.f) + lA * swA;
          mrg_l[2 * t4 + 1] = (w > 0 ? mrg_l[2 * t4 + 1] * sbB : 0.f) + lB * swB;
          mrg_m[2 * t4] = MnA;
          mrg_m[2 * t4 + 1] = MnB;
        }
        if (HAS_V) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {              // (dim 16 j + 8 (i >> 1) + g8, head 2 t4 + (i & 1)): 32 distinct banks
              float* pa = mrg_o + (2 * t4 + (i & 1)) * kMergePitch + 16 * j + 8 * (i >> 1) + g8;
              const float old = w > 0 ? *pa : 0.f;
              *pa = old * ((i & 1) ? sbB : sbA) + o[j][i] * ((i & 1) ? swB : swA);
            }
          }
        }
      }
      __syncthreads();
    }
    // item e = (head e / 16, dims 8 (e % 16) .. + 7) of the CTA's result; kItems items per thread
    {
      constexpr int kItems = kMaxGroup * 16 / kThreads;
      float M[kItems], den[kItems], num[kItems][8];
#pragma unroll
      for (int it = 0; it < kItems; ++it) {
        const int e = it * kThreads + tid, h = e >> 4, d8 = (e & 15) * 8;
        M[it] = mrg_m[h];
        den[it] = mrg_l[h];
        if (HAS_V) {
          const float4 x0 = *reinterpret_cast<const float4*>(mrg_o + h * kMergePitch + d8);
          const float4 x1 = *reinterpret_cast<const float4*>(mrg_o + h * kMergePitch + d8 + 4);
          num[it][0] = x0.x; num[it][1] = x0.y; num[it][2] = x0.z; num[it][3] = x0.w;
          num[it][4] = x1.x; num[it][5] = x1.y; num[it][6] = x1.z; num[it][7] = x1.w;
        }
      }
      // the CTAs that hold a piece of this unit: [c_lo, c_hi]
      int c_lo, c_hi;
      if (split_units) {
        const int per = (uend - ubeg + parts - 1) / parts;
        c_lo = u * parts;
        c_hi = c_lo + (uend - ubeg + per - 1) / per - 1;
      } else {
        c_lo = ubeg / per_cta;
        c_hi = (uend - 1) / per_cta;
      }
      const int64_t head0 = static_cast<int64_t>(u) * G;
      bool finish = true;
      if (merges_in_cluster(split_units, parts)) {
        // The unit's CTAs are one thread-block cluster: CTA 0 of the cluster folds the others'
        // merge buffers into its own through distributed shared memory. Nothing goes through
        // global memory, so nobody waits for the previous kernel. Every CTA of the cluster passes
        // the same two barriers, here or (a CTA without rows) after the loop.
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();                                // every CTA's merged state is in its buffer
        finish = cluster.block_rank() == 0;
        if (finish) {
          const int peers = c_hi - c_lo;               // CTAs 1 .. peers of the cluster hold rows
#pragma unroll 1
          for (int c0 = 1; c0 <= peers; c0 += kMergeRound) {
            float pm[kItems][kMergeRound], pl[kItems][kMergeRound];
            float4 x0[kItems][kMergeRound], x1[kItems][kMergeRound];
#pragma unroll
            for (int r = 0; r < kMergeRound; ++r) {    // a short tail re-reads the last peer (ignored below)
              const float* peer_m = cluster.map_shared_rank(mrg_m, min(c0 + r, peers));
#pragma unroll
              for (int it = 0; it < kItems; ++it) {
                const int e = it * kThreads + tid, h = e >> 4, d8 = (e & 15) * 8;
                pm[it][r] = peer_m[h];
                pl[it][r] = peer_m[8 + h];
                x0[it][r] = x1[it][r] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (HAS_V) {
                  const float4* srcp = reinterpret_cast<const float4*>(peer_m + 16 + h * kMergePitch + d8);
                  x0[it][r] = srcp[0];
                  x1[it][r] = srcp[1];
                }
              }
            }
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
#pragma unroll
              for (int r = 0; r < kMergeRound; ++r) {
                if (c0 + r > peers || pm[it][r] == -INFINITY) continue;
                const float Mn = fmaxf(M[it], pm[it][r]);
                const float so = (M[it] == -INFINITY) ? 0.f : exp2f(M[it] - Mn), sn = exp2f(pm[it][r] - Mn);
                num[it][0] = num[it][0] * so + x0[it][r].x * sn; num[it][1] = num[it][1] * so + x0[it][r].y * sn;
                num[it][2] = num[it][2] * so + x0[it][r].z * sn; num[it][3] = num[it][3] * so + x0[it][r].w * sn;
                num[it][4] = num[it][4] * so + x1[it][r].x * sn; num[it][5] = num[it][5] * so + x1[it][r].y * sn;
                num[it][6] = num[it][6] * so + x1[it][r].z * sn; num[it][7] = num[it][7] * so + x1[it][r].w * sn;
                den[it] = den[it] * so + pl[it][r] * sn;
                M[it] = Mn;
              }
            }
          }
        }
        cluster.sync();                                // no CTA leaves while its buffer may still be read
      } else if (c_lo != c_hi) {                       // the unit is shared with other CTAs
        wait_for_prior_grids();                        // the split workspace may still be in use by the previous kernel
        // a group launch: a range has at most two shared pieces, its first and its last segment
        const int64_t slot = grouped ? 2 * static_cast<int64_t>(blockIdx.x) + (seg_begin == r0 ? 0 : 1) : static_cast<int64_t>(blockIdx.x) + u;
        int* arrivals = a.counters + (grouped ? layer * units + u : u);
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
          const int e = it * kThreads + tid, h = e >> 4, d8 = (e & 15) * 8;
          if (h >= G) continue;
          if (HAS_V) {
            float4* dst = reinterpret_cast<float4*>(a.part_acc + (slot * kMaxGroup + h) * kHeadDim + d8);
            dst[0] = make_float4(num[it][0], num[it][1], num[it][2], num[it][3]);
            dst[1] = make_float4(num[it][4], num[it][5], num[it][6], num[it][7]);
          }
          if ((e & 15) == 0) *reinterpret_cast<float2*>(a.part_ml + (slot * kMaxGroup + h) * 2) = make_float2(M[it], den[it]);
        }
        __threadfence();                               // partial visible before the arrival is counted
        __syncthreads();
        if (tid == 0) {
          const int prev = atomicAdd(arrivals, 1);
          const int last = prev == c_hi - c_lo;
          if (last) *arrivals = 0;                     // ready for the next launch
          *mrg_flag = last;
        }
        __syncthreads();
        finish = *mrg_flag != 0;
        if (finish) {                                  // the last CTA to arrive merges all partials
          __threadfence();
#pragma unroll
          for (int it = 0; it < kItems; ++it) {
            M[it] = -INFINITY;
            den[it] = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) num[it][i] = 0.f;
          }
          // kMergeRound partials of every item of this thread are fetched together, then folded in
#pragma unroll 1
          for (int c0 = c_lo; c0 <= c_hi; c0 += kMergeRound) {
            float2 ml[kItems][kMergeRound];
            float4 x0[kItems][kMergeRound], x1[kItems][kMergeRound];
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
              const int e = it * kThreads + tid, h = e >> 4, d8 = (e & 15) * 8;
              const int hh = h < G ? h : 0;
#pragma unroll
              for (int r = 0; r < kMergeRound; ++r) {  // a short tail re-reads the last partial (ignored below)
                const int cc = min(c0 + r, c_hi);        // CTA cc's piece of this unit: its first segment iff its range starts inside the unit
                const int64_t sl = grouped ? 2 * static_cast<int64_t>(cc) + (cc * per_cta >= ubeg ? 0 : 1) : static_cast<int64_t>(cc) + u;
                ml[it][r] = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (sl * kMaxGroup + hh) * 2));
                x0[it][r] = x1[it][r] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (HAS_V) {
                  const float4* srcp = reinterpret_cast<const float4*>(a.part_acc + (sl * kMaxGroup + hh) * kHeadDim + d8);
                  x0[it][r] = __ldcg(srcp);
                  x1[it][r] = __ldcg(srcp + 1);
                }
              }
            }
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
#pragma unroll
              for (int r = 0; r < kMergeRound; ++r) {
                if (c0 + r > c_hi || ml[it][r].x == -INFINITY) continue;
                const float Mn = fmaxf(M[it], ml[it][r].x);
                const float so = (M[it] == -INFINITY) ? 0.f : exp2f(M[it] - Mn), sn = exp2f(ml[it][r].x - Mn);
                num[it][0] = num[it][0] * so + x0[it][r].x * sn; num[it][1] = num[it][1] * so + x0[it][r].y * sn;
                num[it][2] = num[it][2] * so + x0[it][r].z * sn; num[it][3] = num[it][3] * so + x0[it][r].w * sn;
                num[it][4] = num[it][4] * so + x1[it][r].x * sn; num[it][5] = num[it][5] * so + x1[it][r].y * sn;
                num[it][6] = num[it][6] * so + x1[it][r].z * sn; num[it][7] = num[it][7] * so + x1[it][r].w * sn;
                den[it] = den[it] * so + ml[it][r].y * sn;
                M[it] = Mn;
              }
            }
          }
        }
      }
      if (finish) {
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
          const int e = it * kThreads + tid, h = e >> 4, d8 = (e & 15) * 8;
          if (h >= G) continue;
          if (HAS_V) {
            const float inv = den[it] > 0.f ? 1.f / den[it] : 0.f;
            const int64_t oi = (head0 + h) * kHeadDim + d8;
            void* out_l = static_cast<char*>(a.out) + layer * a.out_layer_bytes;
#pragma unroll
            for (int i = 0; i < 8; i += 2) store_pair(out_l, a.out_is_fp32, oi + i, num[it][i] * inv, num[it][i + 1] * inv);
          }
          if (LOGITS && (e & 15) == 0) {
            a.stats[(head0 + h) * 2 + 0] = M[it];
            a.stats[(head0 + h) * 2 + 1] = den[it];
          }
        }
      }
    }
    seg_begin += seg_rows;
    ++u;
    carried = carry_next;
  }
  cp_async_wait<0>();
  if (r0 >= r1 && merges_in_cluster(split_units, parts)) {
    cg::cluster_group cluster = cg::this_cluster();    // a CTA without rows: the two barriers of the cluster merge
    cluster.sync();
    cluster.sync();
  }
  FASTOCR_TRACE_MARK(5);
#ifdef FASTOCR_TRACE
  if (a.trace != nullptr && lane == 0) {
    a.trace[(blockIdx.x * kAttnWarps + warp) * 16 + 6] = (static_cast<unsigned long long>(trace_wait) << 32) | trace_qk;
    a.trace[(blockIdx.x * kAttnWarps + warp) * 16 + 7] = (static_cast<unsigned long long>(trace_look) << 32) | trace_pv;
  }
#endif

  if ((HAS_IDX || PAGED) && bad_entries != 0 && lane < kBlockTokens) atomicAdd(a.fault_counter, static_cast<unsigned long long>(bad_entries));
  if (bad_lengths != 0) atomicAdd(a.fault_counter, static_cast<unsigned long long>(bad_lengths));

  // A kernel of this library must not complete before its predecessor has (later kernels rely on
  // "my predecessor is done, hence everything before it"). CTAs that wrote only their own output
  // slice did not have to wait; one CTA anchors the chain, the others free their SM slots at once.
  if (blockIdx.x == 0) wait_for_prior_grids();

  // ---- sequences with nothing to attend get zeros (rare; kept off the main path) ---------------
  if (blockIdx.x == 0 && mrg_flag[3] != 0) {           // (never with a plan: it is valid only when no unit is empty)
    for (int e = 0; e < units; ++e) {
      if (prefix_s[e + 1] != prefix_s[e]) continue;
      if (load_geom(a, e / Hkv, HAS_IDX).n_tok != 0) continue;   // not part of this launch: left alone
      wait_for_prior_grids();
      const int64_t head0 = static_cast<int64_t>(e) * G;
      for (int l = 0; l < n_layers; ++l)
        for (int i = tid; i < G * kHeadDim / 2; i += kThreads)
          if (HAS_V) store_pair(static_cast<char*>(a.out) + l * a.out_layer_bytes, a.out_is_fp32, head0 * kHeadDim + 2 * i, 0.f, 0.f);
      for (int i = tid; i < G; i += kThreads)
        if (LOGITS) {
          a.stats[(head0 + i) * 2 + 0] = -INFINITY;
          a.stats[(head0 + i) * 2 + 1] = 0.f;
        }
    }
  }
}

// The set-up of attn_stream_kernel done once for all CTAs of a launch shape: rows per unit, their
// prefix, the way rows are handed out, and per CTA its range, unit and the unit's geometry.
__global__ void __launch_bounds__(kMaxUnits) attn_plan_kernel(const AttnLaunch a, int4* __restrict__ plan_out) {
  __shared__ int prefix_s[kMaxUnits + 1];
  __shared__ int warp_tot[kMaxUnits / 32], warp_max[kMaxUnits / 32];
  wait_for_prior_grids();                              // the previous users of the plan are done
  dependents_may_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Hkv = a.num_kv_heads, units = a.batch * Hkv, grid = a.grid_ctas;
  SeqGeom sg = {0, 0, 0, 0};
  int rows = 0;
  if (tid < units) {
    int bad = 0;
    sg = load_geom(a, tid / Hkv, a.idx != nullptr, bad);
    rows = (sg.n_tok + kRowTokens - 1) / kRowTokens;
    if (bad != 0 && tid % Hkv == 0) atomicAdd(a.fault_counter, static_cast<unsigned long long>(bad));
  }
  int incl = rows, longest = rows;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
    longest = max(longest, __shfl_xor_sync(0xffffffffu, longest, o));
  }
  if (lane == 31) warp_tot[warp] = incl;
  if (lane == 0) warp_max[warp] = longest;
  __syncthreads();
  int before = 0;
  longest = 0;
  for (int w = 0; w < kMaxUnits / 32; ++w) {
    if (w < warp) before += warp_tot[w];
    longest = max(longest, warp_max[w]);
  }
  if (tid < units) prefix_s[tid + 1] = before + incl;
  if (tid == 0) prefix_s[0] = 0;
  const int any_empty = __syncthreads_or(tid < units && rows == 0);
  const int total_rows = prefix_s[units];
  const int parts_rule = split_rule(units, grid, total_rows, longest, true);
  const bool split_units = parts_rule > 0;
  const int parts = max(parts_rule, 1);
  const int per_cta = (total_rows + grid - 1) / grid;
  for (int c = tid; c < grid; c += blockDim.x) {
    int r0 = 0, r1 = 0, u = 0, valid = any_empty ? 0 : 1;
    if (split_units) {
      u = c / parts;
      if (u < units) {
        const int ub = prefix_s[u], ue = prefix_s[u + 1];
        const int per = (ue - ub + parts - 1) / parts;
        r0 = min(ue, ub + (c - u * parts) * per);
        r1 = min(ue, r0 + per);
      } else {
        u = 0;                                         // a CTA without work: an empty range of unit 0
      }
    } else {
      r0 = min(total_rows, c * per_cta);
      r1 = min(total_rows, r0 + per_cta);
      int lo = 0, hi = units;                          // largest u with prefix[u] <= r0
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (prefix_s[mid] <= r0) lo = mid; else hi = mid;
      }
      u = lo;
      if (r1 > prefix_s[u + 1]) valid = 0;             // the range spans several units
      if (r0 >= r1) { u = 0; r0 = r1 = 0; }
    }
    const SeqGeom g = load_geom(a, u / Hkv, a.idx != nullptr);
    int4* rec = plan_out + 4 * static_cast<int64_t>(c);
    rec[0] = make_int4(valid, u, r0, r1);
    rec[1] = make_int4(prefix_s[u], prefix_s[u + 1], split_units ? 1 : 0, parts);
    rec[2] = make_int4(per_cta, total_rows, 0, 0);
    rec[3] = make_int4(g.vs, g.N, g.kept_vis, g.n_tok);
  }
}

constexpr int kFinalizeThreads = 256;

// four tokens per thread (16-byte loads when the layout allows), eight heads' loads in flight
__global__ void __launch_bounds__(kFinalizeThreads) scores_finalize_kernel(
    const float* __restrict__ logits, const float* __restrict__ stats, const int32_t* __restrict__ vis_len,
    int num_q_heads, int n_stride_logits, float* __restrict__ scores, int n_stride) {
  extern __shared__ float st[];                        // [H][2]: max, 1/sum
  wait_for_prior_grids();
  dependents_may_launch();
  const int b = blockIdx.y;
  const int N = min(min(vis_len[b], n_stride), n_stride_logits);
  const int i0 = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (blockIdx.x * blockDim.x * 4 >= N) return;        // the whole CTA is past the end
  for (int i = threadIdx.x; i < num_q_heads; i += blockDim.x) {
    st[2 * i] = stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2];
    st[2 * i + 1] = 1.0f / stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2 + 1];
  }
  __syncthreads();
  if (i0 >= N) return;
  const float* lp = logits + static_cast<int64_t>(b) * num_q_heads * n_stride_logits + i0;
  const bool full = i0 + 4 <= N && (n_stride_logits & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  const uint64_t once = l2_policy_evict_first();
  for (int h0 = 0; h0 < num_q_heads; h0 += 8) {        // summed in head order
    float4 x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      x[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (h0 + j < num_q_heads) {
        const float* src = lp + static_cast<int64_t>(h0 + j) * n_stride_logits;
        if (full) {
          x[j] = load_logit4(src, once);
        } else {
          x[j].x = load_logit(src, once);
          if (i0 + 1 < N) x[j].y = load_logit(src + 1, once);
          if (i0 + 2 < N) x[j].z = load_logit(src + 2, once);
          if (i0 + 3 < N) x[j].w = load_logit(src + 3, once);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (h0 + j < num_q_heads) {
        const float m = st[2 * (h0 + j)], inv = st[2 * (h0 + j) + 1];
        acc[0] = score_add_head(acc[0], x[j].x, m, inv);
        acc[1] = score_add_head(acc[1], x[j].y, m, inv);
        acc[2] = score_add_head(acc[2], x[j].z, m, inv);
        acc[3] = score_add_head(acc[3], x[j].w, m, inv);
      }
    }
  }
  float* out = scores + static_cast<int64_t>(b) * n_stride + i0;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    if (i0 + j < N) out[j] = score_finish(acc[j], num_q_heads);
}

__global__ void __launch_bounds__(1024) image_mass_kernel(const float* __restrict__ scores, int n_stride,
                                                          const int32_t* __restrict__ vis_len, float* __restrict__ mass) {
  __shared__ float red[32];
  wait_for_prior_grids();
  dependents_may_launch();
  const int b = blockIdx.x, N = min(vis_len[b], n_stride);
  float s = 0.f;
  for (int i = threadIdx.x; i < N; i += blockDim.x) s += scores[static_cast<int64_t>(b) * n_stride + i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    s = red[threadIdx.x];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) mass[b] = s;
  }
}

// Cluster sizes (2 .. kMaxPartsPerUnit) the device can schedule for a kernel instance, asked once
// in configure_t; a size it cannot schedule falls back to the merge through global memory.
template <int G, int MODE, bool PAGED>
bool* cluster_ok_table() {
  static bool ok[kMaxPartsPerUnit + 1] = {};
  return ok;
}

template <int G, int MODE, bool PAGED>
cudaError_t launch_partial_t(const AttnLaunch& a, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.grid_ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Smem<MODE != kModeKeys>::total;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  {
    const int c = a.cluster_ctas;
    if (c >= 2 && c <= kMaxPartsPerUnit && a.grid_ctas % c == 0 && cluster_ok_table<G, MODE, PAGED>()[c]) {
      attr[1].id = cudaLaunchAttributeClusterDimension;
      attr[1].val.clusterDim.x = c;
      attr[1].val.clusterDim.y = 1;
      attr[1].val.clusterDim.z = 1;
      cfg.numAttrs = 2;
    }
  }
  const cudaError_t e = cudaLaunchKernelEx(&cfg, attn_stream_kernel<G, MODE, PAGED>, a);
  count_launches(1);
  if (cfg.numAttrs == 2) count_cluster_launches(1);
  return e;
}

template <int G, int MODE>
cudaError_t launch_mode_t(const AttnLaunch& a, cudaStream_t s) {
  return a.page_size > 0 ? launch_partial_t<G, MODE, true>(a, s) : launch_partial_t<G, MODE, false>(a, s);
}

template <int G, int MODE, bool PAGED>
cudaError_t configure_t() {
  cudaError_t e = cudaFuncSetAttribute(attn_stream_kernel<G, MODE, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Smem<MODE != kModeKeys>::total);
  if (e != cudaSuccess) return e;
  // all of the SM's L1/shared array as shared memory: four CTAs must fit
  e = cudaFuncSetAttribute(attn_stream_kernel<G, MODE, PAGED>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
  if (e != cudaSuccess) return e;
  {
    // clusters of more than 8 CTAs need the kernel's consent; which sizes the device can place is asked, not assumed
    const bool big = cudaFuncSetAttribute(attn_stream_kernel<G, MODE, PAGED>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    bool* ok = cluster_ok_table<G, MODE, PAGED>();
    for (int c = 2; c <= kMaxPartsPerUnit; ++c) {
      ok[c] = false;
      if (c > 8 && !big) continue;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(c);
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = Smem<MODE != kModeKeys>::total;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = c;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, attn_stream_kernel<G, MODE, PAGED>, &cfg) == cudaSuccess && n > 0) ok[c] = true;
    }
    (void)cudaGetLastError();                          // a refused size is an answer, not an error
  }
  return cudaSuccess;
}

}  // namespace

#define FASTOCR_FOR_EACH_GROUP(X) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8)

cudaError_t launch_attn_plan(const AttnLaunch& a, int4* plan_out, cudaStream_t s) {
  if (a.batch * a.num_kv_heads > kMaxUnits || a.grid_ctas <= 0) return cudaErrorInvalidValue;
  const cudaError_t e = launch_pdl(attn_plan_kernel, dim3(1), dim3(kMaxUnits), 0, s, a, plan_out);
  count_launches(1);
  return e;
}

cudaError_t launch_attn_partial(const AttnLaunch& a, cudaStream_t s) {
  const int G = a.num_q_heads / a.num_kv_heads;
  // the mode follows from what the launch was given
  const int mode = a.idx != nullptr ? kModePruned : (a.v == nullptr ? kModeKeys : (a.logits != nullptr ? kModeScores : kModeDense));
  if (mode == kModeKeys && a.logits == nullptr) return cudaErrorInvalidValue;
  switch (G) {
#define X(g)                                                      \
  case g:                                                         \
    switch (mode) {                                               \
      case kModePruned: return launch_mode_t<g, kModePruned>(a, s); \
      case kModeScores: return launch_mode_t<g, kModeScores>(a, s); \
      case kModeDense: return launch_mode_t<g, kModeDense>(a, s);   \
      default: return launch_mode_t<g, kModeKeys>(a, s);            \
    }
    FASTOCR_FOR_EACH_GROUP(X)
#undef X
    default:
      return cudaErrorInvalidValue;
  }
}

cudaError_t configure_kernels() {
  cudaError_t e;
  // keep the SMs' shared-memory carve-out where the attention kernel needs it, so that the small
  // kernels in between do not trigger a reconfiguration
  if ((e = cudaFuncSetAttribute(scores_finalize_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(image_mass_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100)) != cudaSuccess) return e;
#define Y(g, m)                                                    \
  if ((e = configure_t<g, m, false>()) != cudaSuccess) return e;   \
  if ((e = configure_t<g, m, true>()) != cudaSuccess) return e;
#define X(g) Y(g, kModePruned) Y(g, kModeScores) Y(g, kModeDense) Y(g, kModeKeys)
  FASTOCR_FOR_EACH_GROUP(X)
#undef X
#undef Y
  return cudaSuccess;
}

#ifdef FASTOCR_TRACE
// debug builds: resident CTAs per SM the runtime grants the 7-head attention kernel
extern "C" int fastocr_debug_occupancy() {
  int n = -1;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, attn_stream_kernel<7, kModeDense, false>, kThreads, Smem<true>::total);
  cudaFuncAttributes fa;
  cudaFuncGetAttributes(&fa, attn_stream_kernel<7, kModeDense, false>);
  return n * 1000 + fa.numRegs;
}
#endif

cudaError_t launch_scores_finalize(const float* logits, const float* stats, const int32_t* vis_len, int32_t batch,
                                   int32_t num_q_heads, int32_t n_stride_logits, int32_t max_vis_len, float* scores,
                                   int32_t n_stride, cudaStream_t s) {
  if (max_vis_len <= 0) return cudaSuccess;
  dim3 grid((max_vis_len + 4 * kFinalizeThreads - 1) / (4 * kFinalizeThreads), batch);
  const cudaError_t e = launch_pdl(scores_finalize_kernel, grid, dim3(kFinalizeThreads), num_q_heads * 2 * sizeof(float), s,
                                   logits, stats, vis_len, num_q_heads, n_stride_logits, scores, n_stride);
  count_launches(1);
  return e;
}

cudaError_t launch_image_mass(const float* scores, int32_t n_stride, const int32_t* vis_len, int32_t batch, float* mass,
                              cudaStream_t s) {
  const cudaError_t e = launch_pdl(image_mass_kernel, dim3(batch), dim3(1024), 0, s, scores, n_stride, vis_len, mass);
  count_launches(1);
  return e;
}

}  // namespace fastocr
