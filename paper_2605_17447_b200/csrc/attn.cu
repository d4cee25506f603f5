// Decode attention kernels for sm_100a: one templated split-KV flash-decode core serves dense
// attention (Eq. 2, focal case), the keys-only scoring pass, and pruned attention over the kept
// set K = T u F (Eq. 2, non-focal case), on contiguous or paged caches.
//
// Work decomposition: CTA = (split c, KV head g, sequence b). The CTA first builds, in shared
// memory, the table of physical cache rows of the tokens it attends (this is the only place where
// dense / pruned / paged differ), then each of its warps streams 16-token blocks of those rows.
//
// Data path: every lane copies, with 16-byte cp.async, exactly the K and V bytes it will later
// need as tensor-core fragments into its own slots of a shared-memory ring (kStages deep; no
// cross-thread hand-off, hence no barrier in the main loop) and reads them back with ld.shared.v4.
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

struct SeqGeom {
  int S, vs, N, kept_vis, n_tok;   // n_tok = number of attended tokens
};

__device__ __forceinline__ SeqGeom load_geom(const AttnLaunch& a, int b) {
  SeqGeom s;
  s.S = a.seq_len[b];
  s.vs = a.vis_start[b];
  s.N = a.vis_len[b];
  if (a.idx != nullptr) {
    int kk = a.kcount[b];
    s.kept_vis = kk < 0 ? 0 : (kk > s.N ? s.N : kk);
  } else {
    s.kept_vis = s.N;
  }
  s.n_tok = s.S - s.N + s.kept_vis;
  return s;
}

// shared-memory carve-up (bytes). A stage holds, per lane, 8 K slots (+ 8 V slots) of 16 bytes.
template <bool HAS_V>
struct Smem {
  static constexpr int kSlots = HAS_V ? 16 : 8;
  static constexpr int kStageBytes = kSlots * 32 * 16;             // per warp
  static constexpr int kRingBytes = kAttnWarps * kStages * kStageBytes;
  static constexpr int kMergeBytes = (kAttnWarps * 16 + kAttnWarps * kMaxGroup * kHeadDim) * 4;
  static constexpr int ring = 0;
  static constexpr int rows = kRingBytes > kMergeBytes ? kRingBytes : kMergeBytes;   // int32 [chunk_tokens]
  static int total(int chunk_tokens) { return rows + chunk_tokens * 4; }
};

template <int G, bool HAS_V>
__global__ void __launch_bounds__(kThreads, 2) attn_partial_kernel(const AttnLaunch a) {
  extern __shared__ __align__(16) unsigned char smem[];
  using L = Smem<HAS_V>;
  const int c = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g8 = lane >> 2, t4 = lane & 3;             // MMA fragment coordinates: group, thread-in-group

  const SeqGeom sg = load_geom(a, b);
  const int start = c * a.chunk_tokens;
  if (start >= sg.n_tok) return;                       // whole CTA leaves together
  const int cnt = min(a.chunk_tokens, sg.n_tok - start);

  // ---- table of physical rows for the attended tokens [start, start + cnt) -------------------
  int32_t* rows_s = reinterpret_cast<int32_t*>(smem + L::rows);
  for (int i = tid; i < cnt; i += kThreads) {
    const int j = start + i;
    int pos = j;
    if (a.idx != nullptr) {                            // kept set: text before | selected image | text after
      if (j >= sg.vs + sg.kept_vis) {
        pos = j - sg.kept_vis + sg.N;
      } else if (j >= sg.vs) {
        int r = a.idx[static_cast<int64_t>(b) * a.k_stride + (j - sg.vs)];
        if (r < 0 || r >= sg.N) {                      // never read outside the image span
          atomicAdd(a.fault_counter, 1ULL);
          r = r < 0 ? 0 : sg.N - 1;
        }
        pos = sg.vs + r;
      }
    }
    int row = pos;
    if (a.page_size > 0) {
      const int page = a.block_table[static_cast<int64_t>(b) * a.max_pages + pos / a.page_size];
      row = page * a.page_size + pos % a.page_size;
    }
    rows_s[i] = row;
  }

  // ---- A fragments of Q: lane (g8, t4) holds head g8, dims 32j + 8 t4 .. + 8 (j = 0..3) -------
  uint32_t qw[4][4];
  {
    const uint4* qp = reinterpret_cast<const uint4*>(a.q) +
                      (static_cast<int64_t>(b) * a.num_q_heads + static_cast<int64_t>(g) * G + g8) * (kHeadDim / 8) + t4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint4 w = make_uint4(0u, 0u, 0u, 0u);
      if (g8 < G) w = __ldg(qp + 4 * j);
      qw[j][0] = w.x; qw[j][1] = w.y; qw[j][2] = w.z; qw[j][3] = w.w;
    }
  }
  __syncthreads();

  const float scale_log2 = a.sm_scale * 1.4426950408889634f;
  const int64_t row_elems = static_cast<int64_t>(a.num_kv_heads) * kHeadDim;
  const int64_t seq_base = a.page_size > 0 ? 0 : static_cast<int64_t>(b) * a.seq_stride_tokens * row_elems;
  const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.k) + seq_base + g * kHeadDim + 8 * t4;
  const __nv_bfloat16* vbase =
      HAS_V ? reinterpret_cast<const __nv_bfloat16*>(a.v) + seq_base + g * kHeadDim + 8 * g8 : nullptr;

  const int n_blocks = (cnt + kBlockTokens - 1) / kBlockTokens;
  const int n_iter = n_blocks > warp ? (n_blocks - warp + kAttnWarps - 1) / kAttnWarps : 0;

  const uint32_t smem_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const uint32_t ring_lane = smem_u32 + L::ring + warp * kStages * L::kStageBytes + lane * 16;

  // Slots of a stage: 0..3 K of token g8 (dims 32j + 8 t4), 4..7 K of token 8 + g8,
  // 8 + 2u + piece: V of token {2 t4, 2 t4 + 1, 8 + 2 t4, 9 + 2 t4}[u], dims 64 piece + 8 g8 .. + 8.
  auto issue = [&](int it) {
    if (it < n_iter) {
      const int tok0 = (warp + it * kAttnWarps) * kBlockTokens;
      const uint32_t dst = ring_lane + (it % kStages) * L::kStageBytes;
      const __nv_bfloat16* ka = kbase + rows_s[min(tok0 + g8, cnt - 1)] * row_elems;
      const __nv_bfloat16* kb = kbase + rows_s[min(tok0 + 8 + g8, cnt - 1)] * row_elems;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        cp_async16(dst + j * 512, ka + 32 * j);
        cp_async16(dst + (4 + j) * 512, kb + 32 * j);
      }
      if (HAS_V) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int tk = tok0 + 2 * t4 + (u & 1) + 8 * (u >> 1);
          const __nv_bfloat16* vr = vbase + rows_s[min(tk, cnt - 1)] * row_elems;
          cp_async16(dst + (8 + 2 * u) * 512, vr);
          cp_async16(dst + (9 + 2 * u) * 512, vr + 64);
        }
      }
    }
    cp_async_commit();
  };

#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) issue(s);

  // O^T accumulators: o[j] is the 16 x 8 tile of dims {64 (j >> 2) + 8 g8 + 2 (j & 3) + (0|1)} x heads;
  // o[j][0..1] = even dim, heads 2 t4, 2 t4 + 1; o[j][2..3] = odd dim, same heads.
  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
  float m_ref = -INFINITY, l_part = 0.f;               // for head g8 (identical in the 4 lanes of a group)
  const bool head_ok = g8 < G;
  const int vis_lo = sg.vs, vis_hi = sg.vs + sg.N;
  float* logit_row = (a.logits != nullptr && head_ok)
                         ? a.logits + (static_cast<int64_t>(b) * a.num_q_heads + g * G + g8) * a.n_stride
                         : nullptr;

  for (int it = 0; it < n_iter; ++it) {
    cp_async_wait<kStages - 2>();
    const uint32_t src = ring_lane + (it % kStages) * L::kStageBytes;
    // ---- S^T = Q K^T for the two 8-token tiles ------------------------------------------------
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 ka = lds128(src + j * 512), kb = lds128(src + (4 + j) * 512);
      mma_bf16(sa, qw[j][0], 0u, qw[j][1], 0u, ka.x, ka.y);
      mma_bf16(sa, qw[j][2], 0u, qw[j][3], 0u, ka.z, ka.w);
      mma_bf16(sb, qw[j][0], 0u, qw[j][1], 0u, kb.x, kb.y);
      mma_bf16(sb, qw[j][2], 0u, qw[j][3], 0u, kb.z, kb.w);
    }
    uint4 vw[4][2];
    if (HAS_V) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        vw[u][0] = lds128(src + (8 + 2 * u) * 512);
        vw[u][1] = lds128(src + (9 + 2 * u) * 512);
      }
    }
    issue(it + kStages - 1);

    // ---- online softmax for head g8, tokens tok0 + {2 t4, 2 t4 + 1, 8 + 2 t4, 9 + 2 t4} ------
    const int tok0 = (warp + it * kAttnWarps) * kBlockTokens;
    float x[4] = {sa[0] * scale_log2, sa[1] * scale_log2, sb[0] * scale_log2, sb[1] * scale_log2};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int tok = tok0 + 2 * t4 + (i & 1) + 8 * (i >> 1);
      const bool valid = head_ok && tok < cnt;
      x[i] = valid ? x[i] : -INFINITY;
      if (logit_row != nullptr && valid) {
        const int pos = start + tok;                   // dense / scoring mode: position == list index
        if (pos >= vis_lo && pos < vis_hi && pos - vis_lo < a.n_stride) logit_row[pos - vis_lo] = x[i];
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
  }
  cp_async_wait<0>();

  // ---- merge inside the warp: the sum of probabilities of head g8 ----------------------------
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
  __syncthreads();                                     // every warp is done with its ring

  // ---- merge across warps (re-using the ring space) and emit the split's partial --------------
  float* m_s = reinterpret_cast<float*>(smem + L::ring);            // [warps][8]
  float* l_s = m_s + kAttnWarps * 8;                                 // [warps][8]
  float* acc_s = l_s + kAttnWarps * 8;                               // [warps][8][128]
  if (t4 == 0) {
    m_s[warp * 8 + g8] = head_ok ? m_ref : -INFINITY;
    l_s[warp * 8 + g8] = head_ok ? l_part : 0.f;
  }
  if (HAS_V) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int d0 = 64 * (j >> 2) + 8 * g8 + 2 * (j & 3);
      float* base = acc_s + (warp * 8 + 2 * t4) * kHeadDim + d0;
      *reinterpret_cast<float2*>(base) = make_float2(o[j][0], o[j][2]);
      *reinterpret_cast<float2*>(base + kHeadDim) = make_float2(o[j][1], o[j][3]);
    }
  }
  __syncthreads();
  const int64_t item = (static_cast<int64_t>(b) * a.num_kv_heads + g) * a.max_chunks + c;
  for (int e = tid; e < G * kHeadDim; e += kThreads) {
    const int h = e / kHeadDim, dd = e % kHeadDim;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, m_s[w * 8 + h]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float mw = m_s[w * 8 + h];
      const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
      den += l_s[w * 8 + h] * sc;
      if (HAS_V) num += acc_s[(w * 8 + h) * kHeadDim + dd] * sc;
    }
    if (HAS_V) a.part_acc[(item * G + h) * kHeadDim + dd] = num;
    if (dd == 0) {
      a.part_ml[(item * G + h) * 2 + 0] = M;
      a.part_ml[(item * G + h) * 2 + 1] = den;
    }
  }
}

// One CTA per (sequence, query head): merge the splits.
__global__ void __launch_bounds__(kHeadDim) attn_combine_kernel(const AttnLaunch a, void* out, int out_is_fp32,
                                                                float* stats) {
  const int h = blockIdx.x, b = blockIdx.y, dd = threadIdx.x;
  const int G = a.num_q_heads / a.num_kv_heads;
  const int g = h / G, hh = h % G;
  const SeqGeom sg = load_geom(a, b);
  const int n_chunks = sg.n_tok > 0 ? (sg.n_tok + a.chunk_tokens - 1) / a.chunk_tokens : 0;
  const int64_t item0 = (static_cast<int64_t>(b) * a.num_kv_heads + g) * a.max_chunks;
  float M = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, a.part_ml[((item0 + c) * G + hh) * 2]);
  float num = 0.f, den = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    const float mc = a.part_ml[((item0 + c) * G + hh) * 2];
    const float sc = (mc == -INFINITY) ? 0.f : exp2f(mc - M);
    den += a.part_ml[((item0 + c) * G + hh) * 2 + 1] * sc;
    if (out != nullptr) num += a.part_acc[((item0 + c) * G + hh) * kHeadDim + dd] * sc;
  }
  if (out != nullptr) {
    const float o = den > 0.f ? num / den : 0.f;
    const int64_t oi = (static_cast<int64_t>(b) * a.num_q_heads + h) * kHeadDim + dd;
    if (out_is_fp32) reinterpret_cast<float*>(out)[oi] = o;
    else reinterpret_cast<__nv_bfloat16*>(out)[oi] = __float2bfloat16_rn(o);
  }
  if (stats != nullptr && dd == 0) {
    stats[(static_cast<int64_t>(b) * a.num_q_heads + h) * 2 + 0] = M;
    stats[(static_cast<int64_t>(b) * a.num_q_heads + h) * 2 + 1] = den;
  }
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
  const int smem = Smem<HAS_V>::total(a.chunk_tokens);
  dim3 grid(a.max_chunks, a.num_kv_heads, a.batch);
  attn_partial_kernel<G, HAS_V><<<grid, kThreads, smem, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

template <int G, bool HAS_V>
cudaError_t configure_t() {
  return cudaFuncSetAttribute(attn_partial_kernel<G, HAS_V>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Smem<HAS_V>::total(kMaxChunk));
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
#define X(g)                                                \
  if ((e = configure_t<g, true>()) != cudaSuccess) return e; \
  if ((e = configure_t<g, false>()) != cudaSuccess) return e;
  FASTOCR_FOR_EACH_GROUP(X)
#undef X
  return cudaSuccess;
}

cudaError_t launch_attn_combine(const AttnLaunch& a, void* out, int out_is_fp32, float* stats, cudaStream_t s) {
  dim3 grid(a.num_q_heads, a.batch);
  attn_combine_kernel<<<grid, kHeadDim, 0, s>>>(a, out, out_is_fp32, stats);
  count_launches(1);
  return cudaGetLastError();
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
