// Decode attention kernels for sm_100a: one templated persistent flash-decode core serves dense
// attention (Eq. 2, focal case), the keys-only scoring pass, and pruned attention over the kept
// set K = T u F (Eq. 2, non-focal case), on contiguous or paged caches.
//
// Work decomposition (stream-K over tokens). All attended tokens of the launch are laid end to end
// in one index space, sequence after sequence, each sequence padded to a multiple of 16 tokens.
// That space is cut into equal ranges, one per "team"; a team is one warp per KV head (so the
// whole 1-2 KB token row is fetched by neighbouring warps at about the same time), and the grid is
// two persistent CTAs of four autonomous warps per SM. Every warp therefore streams the same
// number of 16-token blocks, pays one pipeline prologue per launch, and never meets a CTA barrier
// after set-up. A range may cross sequence boundaries: the warp then finishes the sequence it leaves
// and starts a new one. A sequence covered by one team is normalised and written by that team;
// one shared by several teams is merged by whichever of them arrives last (partials in global
// memory, one atomic arrival counter per sequence and KV head, nobody waits).
//
// Data path: a block's 16 K rows and 16 V rows (256 bytes each) travel HBM -> shared memory with
// 16-byte cp.async, one full row per half-warp per instruction (so every request covers whole
// 128-byte lines), into a per-warp ring (kStages deep; hand-off inside the warp only: one
// __syncwarp per block). Rows are stored with their 16-byte chunks XOR-swizzled so that the
// tensor-core fragment reads (ld.shared.v4, each lane its own chunks) are bank-conflict free.
// Cache rows are located two blocks
// ahead of the copies by lanes 0-15 (one token each): first the logical position (a load from the
// index list for selected image tokens), one block later the physical row (a block-table load for
// paged caches), so neither lookup sits on the critical path.
//
// Arithmetic: with a GQA group of 7 or 8 query heads per KV head, q.K^T and P.V are skinny matrix
// products ([16 tokens x 128] x [128 x 8 heads]); on the fp32 CUDA cores they need more issue slots
// than the HBM stream leaves time for, so both run on the tensor cores as warp-level
// mma.sync.m16n8k16 (bf16 inputs, fp32 accumulation):
//   S^T[head][token] = Q[head][d] . K^T[d][token]   (heads on M, padded to 16; 8 tokens per tile)
//   O^T[d][head]    += V^T[d][token] . P[token][head] (16 dims per tile; 16 tokens on K)
// The accumulator layout of S^T is exactly the B-operand layout P needs, so probabilities never
// leave registers. bf16 products are exact in fp32; P is split into a bf16 high part and a bf16
// remainder (two MMAs) so that the weighted sum keeps about 16 bits of P. The contraction index
// order inside an MMA is free, which lets every fragment be a plain 16-byte row segment: K needs
// no transposition at all, V^T is formed from pairs of rows with two byte-permutes per register.
// The online softmax keeps a per-head running maximum that is raised only when a logit exceeds
// it by more than 2^8, so the rescale branch is rare.
#include "kernels.h"

#include <cuda_bf16.h>

namespace fastocr {
namespace {

constexpr int kStages = 3;
constexpr int kThreads = kAttnWarps * 32;
constexpr int kBlockTokens = 16;        // tokens per warp per pipeline stage
constexpr float kRescaleSlack = 8.0f;   // log2 units
constexpr int kMergeRound = 3;          // partials fetched together by the merging warp

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
  return r;
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

// Programmatic dependent launch: a launch of this kernel may begin while the previous kernel in the
// stream is still draining. dependents_may_launch() lets the next kernel's CTAs be scheduled as
// soon as resources free up; wait_for_prior_grids() blocks until every earlier kernel has finished
// and its writes are visible (a no-op when the launch carried no such attribute).
__device__ __forceinline__ void dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void wait_for_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// two adjacent outputs (even index), bf16 or fp32
__device__ __forceinline__ void store_pair(void* out, int is_fp32, int64_t index, float x, float y) {
  if (is_fp32) *reinterpret_cast<float2*>(reinterpret_cast<float*>(out) + index) = make_float2(x, y);
  else *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(out) + index) = __floats2bfloat162_rn(x, y);
}

// number of attended tokens of sequence b and the pieces needed to enumerate them
struct SeqGeom {
  int vs, N, kept_vis, n_tok;
};
__device__ __forceinline__ SeqGeom load_geom(const AttnLaunch& a, int b) {
  SeqGeom s;
  const int S = a.seq_len[b];
  s.vs = a.vis_start[b];
  s.N = a.vis_len[b];
  if (a.idx != nullptr) {
    const int kk = a.kcount[b];
    s.kept_vis = kk < 0 ? 0 : (kk > s.N ? s.N : kk);
  } else {
    s.kept_vis = s.N;
  }
  s.n_tok = max(S - s.N + s.kept_vis, 0);
  return s;
}

// chunk swizzles of a staged row (16 chunks of 16 bytes): K fragments are read by (token g8,
// chunk 4j + t4), V fragments by (token pair index t4, chunk g8); see the bank analysis in the reads
__device__ __forceinline__ int k_swz(int tok) { return (tok & 1) << 2; }
__device__ __forceinline__ int v_swz(int tok) { return ((tok >> 1) & 3) << 1; }

// shared-memory carve-up (bytes). A stage holds a 16 x 256 B K tile (+ the same for V) per warp.
template <bool HAS_V>
struct Smem {
  static constexpr int kTileBytes = kBlockTokens * kHeadDim * 2;
  static constexpr int kStageBytes = (HAS_V ? 2 : 1) * kTileBytes;   // per warp
  static constexpr int kRingBytes = kAttnWarps * kStages * kStageBytes;
  static constexpr int ring = 0;
  static constexpr int prefix = kRingBytes;                          // int32 [kMaxUnits + 1]
  static constexpr int total = prefix + (kMaxUnits + 1) * 4;
};

// Unit u (a sequence, or a sequence x team-sized slice of its KV heads) -> sequence and first KV head.
__device__ __forceinline__ void unit_to_seq(const AttnLaunch& a, int u, int& b, int& g_base) {
  if (a.units_per_seq == 1) {
    b = u;
    g_base = 0;
  } else {
    b = u / a.units_per_seq;
    g_base = (u - b * a.units_per_seq) * a.team_size;
  }
}

#ifdef FASTOCR_TRACE
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define FASTOCR_TRACE_MARK(slot)                                                                            \
  do {                                                                                                      \
    if (a.trace != nullptr && lane == 0) a.trace[(blockIdx.x * kAttnWarps + warp) * 8 + (slot)] = trace_now(); \
  } while (0)
#else
#define FASTOCR_TRACE_MARK(slot) do { } while (0)
#endif

template <int G, bool HAS_V>
__global__ void __launch_bounds__(kThreads, 2) attn_stream_kernel(const AttnLaunch a) {
  extern __shared__ __align__(16) unsigned char smem[];
  using L = Smem<HAS_V>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g8 = lane >> 2, t4 = lane & 3;             // MMA fragment coordinates: group, thread-in-group
  const int units = a.batch * a.units_per_seq;

  FASTOCR_TRACE_MARK(0);
  // Everything read before the first wait_for_prior_grids() (lengths, index list, queries, cache)
  // must not have been produced by the kernel launched just before this one; the host says so.
  if (a.wait_at_start) wait_for_prior_grids();
  dependents_may_launch();
  // ---- set-up: padded token prefix over units (warp 0), the only CTA barrier of the kernel -----
  int* prefix_s = reinterpret_cast<int*>(smem + L::prefix);
  if (warp == 0) {
    int carry = 0;
    for (int u0 = 0; u0 < units; u0 += 32) {
      const int u = u0 + lane;
      int n = 0;
      if (u < units) {
        int b, gb;
        unit_to_seq(a, u, b, gb);
        n = (load_geom(a, b).n_tok + kBlockTokens - 1) & ~(kBlockTokens - 1);
      }
      int incl = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (u < units) prefix_s[u] = carry + incl - n;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) prefix_s[units] = carry;
  }
  __syncthreads();
  FASTOCR_TRACE_MARK(1);
  const int total_tok = prefix_s[units];
  const int teams = (gridDim.x * kAttnWarps) / a.team_size;
  const int per_team = (((total_tok + teams - 1) / teams) + kBlockTokens - 1) & ~(kBlockTokens - 1);
  if (blockIdx.x == 0) {                               // sequences with nothing to attend: zeros
    for (int u = 0; u < units; ++u) {
      if (prefix_s[u + 1] != prefix_s[u]) continue;
      wait_for_prior_grids();
      int b, gb;
      unit_to_seq(a, u, b, gb);
      const int64_t head0 = static_cast<int64_t>(b) * a.num_q_heads + static_cast<int64_t>(gb) * G;
      for (int e = tid; e < a.team_size * G * kHeadDim / 2; e += kThreads)
        if (HAS_V) store_pair(a.out, a.out_is_fp32, head0 * kHeadDim + 2 * e, 0.f, 0.f);
      for (int e = tid; e < a.team_size * G; e += kThreads)
        if (a.stats != nullptr) {
          a.stats[(head0 + e) * 2 + 0] = -INFINITY;
          a.stats[(head0 + e) * 2 + 1] = 0.f;
        }
    }
  }
  const int wglobal = blockIdx.x * kAttnWarps + warp;
  const int team = wglobal / a.team_size, team_lane = wglobal - team * a.team_size;
  const int r0 = team * per_team;
  const int r1 = min(total_tok, r0 + per_team);
  if (per_team == 0 || r0 >= r1) return;               // nothing for this warp (no barrier follows)
  const int n_blocks = (r1 - r0) / kBlockTokens;

  const float scale_log2 = a.sm_scale * 1.4426950408889634f;
  const int64_t row_elems = static_cast<int64_t>(a.num_kv_heads) * kHeadDim;
  const int64_t seq_elems = a.page_size > 0 ? 0 : a.seq_stride_tokens * row_elems;
  const int c16 = lane & 15, half = lane >> 4;          // copy role: chunk of a row, which row of a pair
  const __nv_bfloat16* kptr = reinterpret_cast<const __nv_bfloat16*>(a.k) + 8 * c16;
  const __nv_bfloat16* vptr = HAS_V ? reinterpret_cast<const __nv_bfloat16*>(a.v) + 8 * c16 : nullptr;
  const uint32_t smem_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const uint32_t ring_warp = smem_u32 + L::ring + warp * kStages * L::kStageBytes;

  // ---- block descriptors: a cursor walks the range; a 5-deep register FIFO feeds the stages ----
  // stage P (block n+4): logical position of token `lane` (< 16) of the block
  // stage R (block n+3): physical row of that token
  // stage I (block n+2): cp.async of the block's K/V fragments
  // stage C (block n):   MMAs, softmax, partial flush
  int cur_u = 0, cur_end = 0;                          // cursor: unit containing the next offset
  {
    int lo = 0, hi = units;                            // largest u with prefix[u] <= r0
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (prefix_s[mid] <= r0) lo = mid; else hi = mid;
    }
    cur_u = lo;
    while (prefix_s[cur_u + 1] <= r0) ++cur_u;         // skip empty units
    cur_end = prefix_s[cur_u + 1];
  }
  int cur_b, cur_gb;
  unit_to_seq(a, cur_u, cur_b, cur_gb);
  SeqGeom cur_geom = load_geom(a, cur_b);

  int fu[5], fj[5], fb[5], fvs[5], fN[5];              // unit, first token within unit, sequence, image span
#pragma unroll
  for (int i = 0; i < 5; ++i) { fu[i] = -1; fj[i] = 0; fb[i] = 0; fvs[i] = 0; fN[i] = 0; }
  int pos_p = 0, row_p = 0;                            // lanes 0..15: position (block n+4 -> n+3), row (n+3 -> n+2)
  bool idx_p = false;                                  // pos_p is a raw index-list entry

  // Describe block n (if it exists) and start its position lookup. For a selected image token the
  // value returned is the raw entry of the index list and `from_idx` is set: nothing may depend on
  // the loaded value here, it is checked and turned into a position one block later (stage_row).
  auto stage_pos = [&](int n, int& du, int& dj, int& db, int& dvs, int& dN, bool& from_idx) -> int {
    from_idx = false;
    if (n >= n_blocks) { du = -1; return 0; }
    const int off = r0 + n * kBlockTokens;
    while (off >= cur_end) {
      ++cur_u;
      cur_end = prefix_s[cur_u + 1];
      if (off < cur_end) {
        unit_to_seq(a, cur_u, cur_b, cur_gb);
        cur_geom = load_geom(a, cur_b);
      }
    }
    du = cur_u;
    dj = off - prefix_s[cur_u];
    db = cur_b;
    dvs = cur_geom.vs;
    dN = cur_geom.N;
    int pos = 0;
    if (lane < kBlockTokens) {
      const int j = min(dj + lane, cur_geom.n_tok - 1);
      pos = j;
      if (a.idx != nullptr) {                          // kept set: text before | selected image | text after
        if (j >= cur_geom.vs + cur_geom.kept_vis) {
          pos = j - cur_geom.kept_vis + cur_geom.N;
        } else if (j >= cur_geom.vs) {
          pos = __ldg(a.idx + static_cast<int64_t>(cur_b) * a.k_stride + (j - cur_geom.vs));
          from_idx = true;
        }
      }
    }
    return pos;
  };
  auto stage_row = [&](int du, int db, int dvs, int dN, bool from_idx, int pos) -> int {
    if (du < 0 || lane >= kBlockTokens) return pos;
    if (from_idx) {
      if (pos < 0 || pos >= dN) {                      // never read outside the image span
        atomicAdd(a.fault_counter, 1ULL);
        pos = pos < 0 ? 0 : dN - 1;
      }
      pos += dvs;
    }
    if (a.page_size == 0) return pos;
    const int page = __ldg(a.block_table + static_cast<int64_t>(db) * a.max_pages + pos / a.page_size);
    return page * a.page_size + pos % a.page_size;
  };
  auto stage_issue = [&](int n, int du, int db, int row) {
    if (du >= 0) {
      int b_unused, gb;
      unit_to_seq(a, du, b_unused, gb);
      const int64_t base = db * seq_elems + static_cast<int64_t>(gb + team_lane) * kHeadDim;
      const uint32_t dst = ring_warp + (n % kStages) * L::kStageBytes;
#pragma unroll
      for (int i = 0; i < 8; ++i) {                    // rows 2i (lanes 0-15) and 2i + 1 (lanes 16-31)
        const int tok = 2 * i + half;
        const int64_t roff = base + __shfl_sync(0xffffffffu, row, tok) * row_elems;
        cp_async16(dst + tok * 256 + ((c16 ^ k_swz(tok)) << 4), kptr + roff);
        if (HAS_V) cp_async16(dst + L::kTileBytes + tok * 256 + ((c16 ^ v_swz(tok)) << 4), vptr + roff);
      }
    }
    cp_async_commit();
  };

  // ---- prologue: positions of blocks 0..3, rows of 0..2, copies of 0..1 -------------------------
  bool idx0, idx1, idx2;
  int pos0 = stage_pos(0, fu[0], fj[0], fb[0], fvs[0], fN[0], idx0);
  int pos1 = stage_pos(1, fu[1], fj[1], fb[1], fvs[1], fN[1], idx1);
  int pos2 = stage_pos(2, fu[2], fj[2], fb[2], fvs[2], fN[2], idx2);
  pos_p = stage_pos(3, fu[3], fj[3], fb[3], fvs[3], fN[3], idx_p);
  {
    const int row0 = stage_row(fu[0], fb[0], fvs[0], fN[0], idx0, pos0);
    const int row1 = stage_row(fu[1], fb[1], fvs[1], fN[1], idx1, pos1);
    row_p = stage_row(fu[2], fb[2], fvs[2], fN[2], idx2, pos2);
    stage_issue(0, fu[0], fb[0], row0);
    stage_issue(1, fu[1], fb[1], row1);
  }
  FASTOCR_TRACE_MARK(2);

  // ---- per-unit state ----------------------------------------------------------------------------
  uint32_t qw[4][4];                                   // A fragments of Q: head g8, dims 32j + 8 t4 .. + 8
  float o[8][4];                                       // O^T tiles: dims {64 (j>>2) + 8 g8 + 2 (j&3) + (0|1)} x heads {2 t4, 2 t4 + 1}
  float m_ref = -INFINITY, l_part = 0.f;               // head g8 (identical in the 4 lanes of a group)
  const bool head_ok = g8 < G;
  int act_u = -1, act_b = 0, act_g = 0, act_ntok = 0, act_vs = 0, act_N = 0;
  float* logit_row = nullptr;

  auto begin_unit = [&](int u, int b) {
    int b2, gb;
    unit_to_seq(a, u, b2, gb);
    act_u = u;
    act_b = b;
    act_g = gb + team_lane;
    const SeqGeom sg = load_geom(a, b);
    act_ntok = sg.n_tok; act_vs = sg.vs; act_N = sg.N;
    const uint4* qp = reinterpret_cast<const uint4*>(a.q) +
                      (static_cast<int64_t>(b) * a.num_q_heads + static_cast<int64_t>(act_g) * G + g8) * (kHeadDim / 8) + t4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint4 w = make_uint4(0u, 0u, 0u, 0u);
      if (head_ok) w = __ldg(qp + 4 * j);
      qw[j][0] = w.x; qw[j][1] = w.y; qw[j][2] = w.z; qw[j][3] = w.w;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
    m_ref = -INFINITY;
    l_part = 0.f;
    logit_row = (a.logits != nullptr && head_ok)
                    ? a.logits + (static_cast<int64_t>(b) * a.num_q_heads + act_g * G + g8) * a.n_stride
                    : nullptr;
  };
  // Leaving a sequence. If its whole (padded) token range lies inside this team's range the warp
  // normalises and writes the result itself. Otherwise it stores its partial (slot (team + unit) *
  // team_size + lane-in-team), bumps the (unit, KV head) arrival counter, and the warp that arrives
  // last merges all partials of that (unit, KV head): no waiting anywhere.
  auto end_unit = [&]() {
    wait_for_prior_grids();                            // results and the shared workspace are written from here on
    float l = l_part;
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    const int ubeg = prefix_s[act_u], uend = prefix_s[act_u + 1];
    const int t_lo = ubeg / per_team, t_hi = (uend - 1) / per_team;
    const int64_t head0 = static_cast<int64_t>(act_b) * a.num_q_heads + static_cast<int64_t>(act_g) * G;
    if (t_lo == t_hi) {
      if (t4 == 0 && head_ok && a.stats != nullptr) {
        a.stats[(head0 + g8) * 2 + 0] = m_ref;
        a.stats[(head0 + g8) * 2 + 1] = l;
      }
      if (HAS_V) {
        const float l0 = __shfl_sync(0xffffffffu, l, 8 * t4), l1 = __shfl_sync(0xffffffffu, l, 8 * t4 + 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int d0 = 64 * (j >> 2) + 8 * g8 + 2 * (j & 3);
          if (2 * t4 < G) store_pair(a.out, a.out_is_fp32, (head0 + 2 * t4) * kHeadDim + d0,
                                     l0 > 0.f ? o[j][0] / l0 : 0.f, l0 > 0.f ? o[j][2] / l0 : 0.f);
          if (2 * t4 + 1 < G) store_pair(a.out, a.out_is_fp32, (head0 + 2 * t4 + 1) * kHeadDim + d0,
                                         l1 > 0.f ? o[j][1] / l1 : 0.f, l1 > 0.f ? o[j][3] / l1 : 0.f);
        }
      }
      return;
    }
    const int64_t slot = (static_cast<int64_t>(team) + act_u) * a.team_size + team_lane;
    if (t4 == 0 && head_ok) {
      a.part_ml[(slot * kMaxGroup + g8) * 2 + 0] = m_ref;
      a.part_ml[(slot * kMaxGroup + g8) * 2 + 1] = l;
    }
    if (HAS_V) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int d0 = 64 * (j >> 2) + 8 * g8 + 2 * (j & 3);
        float* base = a.part_acc + (slot * kMaxGroup + 2 * t4) * kHeadDim + d0;
        if (2 * t4 < G) *reinterpret_cast<float2*>(base) = make_float2(o[j][0], o[j][2]);
        if (2 * t4 + 1 < G) *reinterpret_cast<float2*>(base + kHeadDim) = make_float2(o[j][1], o[j][3]);
      }
    }
    __threadfence();                                   // partial visible before the arrival is counted
    __syncwarp();
    int* counter = a.counters + act_u * a.team_size + team_lane;
    int prev = 0;
    if (lane == 0) prev = atomicAdd(counter, 1);
    prev = __shfl_sync(0xffffffffu, prev, 0);
    if (prev != t_hi - t_lo) return;                   // someone else arrives later and merges
    if (lane == 0) *counter = 0;                       // ready for the next launch
    __threadfence();
    // lane owns dims 4 lane .. 4 lane + 3 of every head; kMergeRound partials per round, all loads of a
    // round issued before any is used (the merge costs one memory latency per round)
    float M[G], den[G];
    float4 num[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
      M[h] = -INFINITY;
      den[h] = 0.f;
      num[h] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int t0 = t_lo; t0 <= t_hi; t0 += kMergeRound) {
      float2 ml[kMergeRound][G];
      float4 acc[kMergeRound][G];
#pragma unroll
      for (int r = 0; r < kMergeRound; ++r) {
        const int t = min(t0 + r, t_hi);               // an odd tail re-reads the last partial (ignored below)
        const int64_t sl = (static_cast<int64_t>(t) + act_u) * a.team_size + team_lane;
#pragma unroll
        for (int h = 0; h < G; ++h) {
          ml[r][h] = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (sl * kMaxGroup + h) * 2));
          acc[r][h] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (HAS_V) acc[r][h] = __ldcg(reinterpret_cast<const float4*>(a.part_acc + (sl * kMaxGroup + h) * kHeadDim) + lane);
        }
      }
#pragma unroll
      for (int r = 0; r < kMergeRound; ++r) {
        if (t0 + r > t_hi) continue;
#pragma unroll
        for (int h = 0; h < G; ++h) {
          if (ml[r][h].x == -INFINITY) continue;
          const float Mn = fmaxf(M[h], ml[r][h].x);
          const float so = (M[h] == -INFINITY) ? 0.f : exp2f(M[h] - Mn), sn = exp2f(ml[r][h].x - Mn);
          num[h].x = num[h].x * so + acc[r][h].x * sn; num[h].y = num[h].y * so + acc[r][h].y * sn;
          num[h].z = num[h].z * so + acc[r][h].z * sn; num[h].w = num[h].w * so + acc[r][h].w * sn;
          den[h] = den[h] * so + ml[r][h].y * sn;
          M[h] = Mn;
        }
      }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      if (HAS_V) {
        const int64_t oi = (head0 + h) * kHeadDim + 4 * lane;
        const float inv = den[h] > 0.f ? 1.f / den[h] : 0.f;
        store_pair(a.out, a.out_is_fp32, oi, num[h].x * inv, num[h].y * inv);
        store_pair(a.out, a.out_is_fp32, oi + 2, num[h].z * inv, num[h].w * inv);
      }
      if (lane == 0 && a.stats != nullptr) {
        a.stats[(head0 + h) * 2 + 0] = M[h];
        a.stats[(head0 + h) * 2 + 1] = den[h];
      }
    }
  };

  for (int n = 0; n < n_blocks; ++n) {
    if (fu[0] != act_u) {                              // the range enters a new sequence
      if (act_u >= 0) end_unit();
      begin_unit(fu[0], fb[0]);
    }
    cp_async_wait<kStages - 2>();
    __syncwarp();                                      // every lane's copies of this block have landed
    if (n == 0) FASTOCR_TRACE_MARK(3);
    const uint32_t src = ring_warp + (n % kStages) * L::kStageBytes;
    // ---- S^T = Q K^T for the two 8-token tiles ------------------------------------------------
    // lane (g8, t4) reads chunk 4j + t4 of rows g8 and 8 + g8: per 8-lane phase two rows whose
    // swizzles differ in bit 2, i.e. eight distinct 16-byte bank groups
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t krow = src + g8 * 256;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t coff = ((4 * j + t4) ^ k_swz(g8)) << 4;        // k_swz(8 + g8) == k_swz(g8)
      const uint4 ka = lds128(krow + coff), kb = lds128(krow + 8 * 256 + coff);
      mma_bf16(sa, qw[j][0], 0u, qw[j][1], 0u, ka.x, ka.y);
      mma_bf16(sa, qw[j][2], 0u, qw[j][3], 0u, ka.z, ka.w);
      mma_bf16(sb, qw[j][0], 0u, qw[j][1], 0u, kb.x, kb.y);
      mma_bf16(sb, qw[j][2], 0u, qw[j][3], 0u, kb.z, kb.w);
    }
    uint4 vw[4][2];
    if (HAS_V) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {                    // rows {2 t4, 2 t4 + 1, 8 + 2 t4, 9 + 2 t4}, chunks g8 and 8 + g8
        const int tk = 2 * t4 + (u & 1) + 8 * (u >> 1);
        const uint32_t vrow = src + L::kTileBytes + tk * 256;
        vw[u][0] = lds128(vrow + ((g8 ^ v_swz(tk)) << 4));
        vw[u][1] = lds128(vrow + (((8 + g8) ^ v_swz(tk)) << 4));
      }
    }
    // ---- keep the look-ahead stages moving ----------------------------------------------------
    stage_issue(n + 2, fu[2], fb[2], row_p);
    row_p = stage_row(fu[3], fb[3], fvs[3], fN[3], idx_p, pos_p);
    pos_p = stage_pos(n + 4, fu[4], fj[4], fb[4], fvs[4], fN[4], idx_p);

    // ---- online softmax for head g8, tokens j0 + {2 t4, 2 t4 + 1, 8 + 2 t4, 9 + 2 t4} ---------
    const int j0 = fj[0];
    float x[4] = {sa[0] * scale_log2, sa[1] * scale_log2, sb[0] * scale_log2, sb[1] * scale_log2};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int tok = j0 + 2 * t4 + (i & 1) + 8 * (i >> 1);         // index in the sequence's attended list
      const bool valid = head_ok && tok < act_ntok;
      x[i] = valid ? x[i] : -INFINITY;
      if (logit_row != nullptr && valid) {             // dense / scoring mode: position == list index
        const int rel = tok - act_vs;
        if (rel >= 0 && rel < act_N && rel < a.n_stride) logit_row[rel] = x[i];
      }
    }
    float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    if (__any_sync(0xffffffffu, mx > m_ref + kRescaleSlack)) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const bool raise = mx > m_ref + kRescaleSlack;
      const float alpha = raise ? fast_exp2(m_ref - mx) : 1.f;     // m_ref = -inf gives 0
      if (raise) m_ref = mx;
      l_part *= alpha;
      if (HAS_V) {
        const float a0 = __shfl_sync(0xffffffffu, alpha, 8 * t4);       // head 2 t4 lives in group 2 t4
        const float a1 = __shfl_sync(0xffffffffu, alpha, 8 * t4 + 4);   // head 2 t4 + 1
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          o[j][0] *= a0; o[j][1] *= a1; o[j][2] *= a0; o[j][3] *= a1;
        }
      }
    }
    float p[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      p[i] = (x[i] == -INFINITY) ? 0.f : fast_exp2(x[i] - m_ref);
      l_part += p[i];
    }

    if (HAS_V) {
      // B fragments of P (tokens on K, head g8 on N): high bf16 part and remainder
      const uint32_t ph0 = pack_bf16(p[0], p[1]), ph1 = pack_bf16(p[2], p[3]);
      const uint32_t pl0 = pack_bf16(p[0] - __uint_as_float(ph0 << 16), p[1] - __uint_as_float(ph0 & 0xffff0000u));
      const uint32_t pl1 = pack_bf16(p[2] - __uint_as_float(ph1 << 16), p[3] - __uint_as_float(ph1 & 0xffff0000u));
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int piece = j >> 2, i = j & 3;
        const uint32_t w0 = (&vw[0][piece].x)[i], w1 = (&vw[1][piece].x)[i];
        const uint32_t w2 = (&vw[2][piece].x)[i], w3 = (&vw[3][piece].x)[i];
        // A fragment of V^T: rows = (even dim, odd dim), columns = token pairs
        const uint32_t a0 = __byte_perm(w0, w1, 0x5410), a1 = __byte_perm(w0, w1, 0x7632);
        const uint32_t a2 = __byte_perm(w2, w3, 0x5410), a3 = __byte_perm(w2, w3, 0x7632);
        mma_bf16(o[j], a0, a1, a2, a3, ph0, ph1);
        mma_bf16(o[j], a0, a1, a2, a3, pl0, pl1);
      }
    }
    // ---- advance the descriptor FIFO ----------------------------------------------------------
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      fu[i] = fu[i + 1]; fj[i] = fj[i + 1]; fb[i] = fb[i + 1]; fvs[i] = fvs[i + 1]; fN[i] = fN[i + 1];
    }
  }
  cp_async_wait<0>();
  FASTOCR_TRACE_MARK(4);
  if (act_u >= 0) end_unit();
  FASTOCR_TRACE_MARK(5);
}

constexpr int kFinalizeThreads = 256;

__global__ void __launch_bounds__(kFinalizeThreads) scores_finalize_kernel(
    const float* __restrict__ logits, const float* __restrict__ stats, const int32_t* __restrict__ vis_len,
    int num_q_heads, int n_stride_logits, float* __restrict__ scores, int n_stride) {
  extern __shared__ float st[];                        // [H][2]: max, 1/sum
  const int b = blockIdx.y;
  const int N = vis_len[b];
  for (int i = threadIdx.x; i < num_q_heads; i += blockDim.x) {
    st[2 * i] = stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2];
    st[2 * i + 1] = 1.0f / stats[(static_cast<int64_t>(b) * num_q_heads + i) * 2 + 1];
  }
  __syncthreads();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N || i >= n_stride || i >= n_stride_logits) return;
  const float* lp = logits + static_cast<int64_t>(b) * num_q_heads * n_stride_logits + i;
  float s = 0.f;
  for (int h = 0; h < num_q_heads; ++h) s += exp2f(lp[static_cast<int64_t>(h) * n_stride_logits] - st[2 * h]) * st[2 * h + 1];
  scores[static_cast<int64_t>(b) * n_stride + i] = s / static_cast<float>(num_q_heads);
}

__global__ void __launch_bounds__(1024) image_mass_kernel(const float* __restrict__ scores, int n_stride,
                                                          const int32_t* __restrict__ vis_len, float* __restrict__ mass) {
  __shared__ float red[32];
  const int b = blockIdx.x, N = vis_len[b];
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

template <int G, bool HAS_V>
cudaError_t launch_partial_t(const AttnLaunch& a, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.grid_ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Smem<HAS_V>::total;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, attn_stream_kernel<G, HAS_V>, a);
  count_launches(1);
  return e;
}

template <int G, bool HAS_V>
cudaError_t configure_t() {
  return cudaFuncSetAttribute(attn_stream_kernel<G, HAS_V>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Smem<HAS_V>::total);
}

}  // namespace

#define FASTOCR_FOR_EACH_GROUP(X) X(1) X(2) X(4) X(7) X(8)

cudaError_t launch_attn_partial(const AttnLaunch& a, cudaStream_t s) {
  const int G = a.num_q_heads / a.num_kv_heads;
  const bool has_v = a.v != nullptr;
  switch (G) {
#define X(g) \
  case g:    \
    return has_v ? launch_partial_t<g, true>(a, s) : launch_partial_t<g, false>(a, s);
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
#define X(g)                                                \
  if ((e = configure_t<g, true>()) != cudaSuccess) return e; \
  if ((e = configure_t<g, false>()) != cudaSuccess) return e;
  FASTOCR_FOR_EACH_GROUP(X)
#undef X
  return cudaSuccess;
}

cudaError_t launch_scores_finalize(const float* logits, const float* stats, const int32_t* vis_len, int32_t batch,
                                   int32_t num_q_heads, int32_t n_stride_logits, int32_t max_vis_len, float* scores,
                                   int32_t n_stride, cudaStream_t s) {
  if (max_vis_len <= 0) return cudaSuccess;
  dim3 grid((max_vis_len + kFinalizeThreads - 1) / kFinalizeThreads, batch);
  scores_finalize_kernel<<<grid, kFinalizeThreads, num_q_heads * 2 * sizeof(float), s>>>(
      logits, stats, vis_len, num_q_heads, n_stride_logits, scores, n_stride);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_image_mass(const float* scores, int32_t n_stride, const int32_t* vis_len, int32_t batch, float* mass,
                              cudaStream_t s) {
  image_mass_kernel<<<batch, 1024, 0, s>>>(scores, n_stride, vis_len, mass);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace fastocr
