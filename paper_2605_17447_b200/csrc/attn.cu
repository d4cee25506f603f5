// Decode attention kernels for sm_100a: one templated split-KV flash-decode core serves dense
// attention (Eq. 2, focal case), the keys-only scoring pass, and pruned attention over the kept
// set K = T u F (Eq. 2, non-focal case), on contiguous or paged caches.
//
// Work decomposition: CTA = (split c, KV head g, sequence b). The CTA first builds, in shared
// memory, the table of physical cache rows of the tokens it attends (this is the only place where
// dense / pruned / paged differ), then its warps stream those rows.
//
// Data path: each lane owns 16 bytes (8 bf16) of a 256-byte K or V row; 16 lanes cover a row, so a
// warp handles two tokens side by side and four tokens per pipeline stage. Rows travel
// HBM -> shared memory with 16-byte cp.async into a per-lane ring (kStages deep, no cross-thread
// hand-off, hence no barrier in the main loop) and are consumed with ld.shared.v4.
// Arithmetic: fp32 throughout, issued as packed fma.rn.f32x2 so that the FMA pipe, not the issue
// port, is the limit; one K row is dotted with all G query heads of the group while in registers.
// Partial dot products are combined across the 16 lanes with a reduce-scatter (15 shuffles per 16
// values) that leaves each (token, head) logit in exactly one lane, which applies the online
// softmax; probabilities are handed back to all lanes through a 128-byte shared-memory slot.
// The running maximum is only raised when a logit exceeds it by more than 2^8 (the accumulators
// stay in range and the rescale branch is rare).
#include "kernels.h"

#include <cuda_bf16.h>

namespace fastocr {
namespace {

constexpr int kStages = 6;
constexpr int kThreads = kAttnWarps * 32;
constexpr float kRescaleSlack = 8.0f;   // log2 units

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 fmul2(u64 a, u64 b) {
  u64 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// two bf16 packed in a 32-bit word -> (low element, high element) widened exactly to fp32
__device__ __forceinline__ u64 widen2(uint32_t w) {
  return pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
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

// shared-memory carve-up (bytes)
template <bool HAS_V>
struct Smem {
  static constexpr int kSlots = HAS_V ? 4 : 2;
  static constexpr int kRingBytes = kAttnWarps * kStages * kSlots * 32 * 16;
  static constexpr int kProbBytes = kAttnWarps * 2 * 32 * 4;
  static constexpr int ring = 0;
  static constexpr int prob = kRingBytes;
  static constexpr int rows = kRingBytes + kProbBytes;       // int32 [chunk_tokens]
  static int total(int chunk_tokens) { return rows + chunk_tokens * 4; }
};

template <int G, bool HAS_V>
__global__ void __launch_bounds__(kThreads, 3) attn_partial_kernel(const AttnLaunch a) {
  extern __shared__ __align__(16) unsigned char smem[];
  using L = Smem<HAS_V>;
  const int c = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, l16 = lane & 15, half = lane >> 4;

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

  // ---- queries of this KV group, pre-scaled to the log2 domain, as f32x2 pairs ----------------
  u64 q2[G][4];
  {
    const float qs = a.sm_scale * 1.4426950408889634f;
    const uint4* qp = reinterpret_cast<const uint4*>(a.q) +
                      (static_cast<int64_t>(b) * a.num_q_heads + static_cast<int64_t>(g) * G) * (kHeadDim / 8) + l16;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const uint4 w = __ldg(qp + h * (kHeadDim / 8));
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        q2[h][i] = pack2(__uint_as_float(ww[i] << 16) * qs, __uint_as_float(ww[i] & 0xffff0000u) * qs);
      }
    }
  }
  __syncthreads();

  const int64_t row_elems = static_cast<int64_t>(a.num_kv_heads) * kHeadDim;
  const int64_t seq_base = a.page_size > 0 ? 0 : static_cast<int64_t>(b) * a.seq_stride_tokens * row_elems;
  const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.k) + seq_base + g * kHeadDim + l16 * 8;
  const __nv_bfloat16* vbase =
      HAS_V ? reinterpret_cast<const __nv_bfloat16*>(a.v) + seq_base + g * kHeadDim + l16 * 8 : nullptr;

  const int n_quads = (cnt + kQuad - 1) / kQuad;
  const int n_iter = n_quads > warp ? (n_quads - warp + kAttnWarps - 1) / kAttnWarps : 0;

  const uint32_t smem_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const uint32_t ring_lane = smem_u32 + L::ring + (warp * kStages * L::kSlots * 32 + lane) * 16;
  float* prob_s = reinterpret_cast<float*>(smem + L::prob) + warp * 64;

  auto issue = [&](int it) {
    if (it < n_iter) {
      const int t0 = (warp + it * kAttnWarps) * kQuad + half * 2;
      const int r0 = rows_s[min(t0, cnt - 1)];
      const int r1 = rows_s[min(t0 + 1, cnt - 1)];
      const uint32_t dst = ring_lane + (it % kStages) * (L::kSlots * 32 * 16);
      cp_async16(dst, kbase + r0 * row_elems);
      cp_async16(dst + 512, kbase + r1 * row_elems);
      if (HAS_V) {
        cp_async16(dst + 1024, vbase + r0 * row_elems);
        cp_async16(dst + 1536, vbase + r1 * row_elems);
      }
    }
    cp_async_commit();
  };

#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) issue(s);

  // online-softmax state. Owner lanes (one per (token-in-pair, head)) keep m_ref / l_part.
  u64 acc2[G][4];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc2[h][i] = 0ULL;
  float m_ref = -INFINITY, l_part = 0.f;
  const int own_h = l16 & 7, own_tt = l16 >> 3;
  const bool own_head_ok = own_h < G;
  const int vis_lo = sg.vs, vis_hi = sg.vs + sg.N;
  float* logit_row = (a.logits != nullptr && own_head_ok)
                         ? a.logits + (static_cast<int64_t>(b) * a.num_q_heads + g * G + own_h) * a.n_stride
                         : nullptr;

  for (int it = 0; it < n_iter; ++it) {
    cp_async_wait<kStages - 2>();
    const uint32_t src = ring_lane + (it % kStages) * (L::kSlots * 32 * 16);
    const uint4 k0 = lds128(src), k1 = lds128(src + 512);
    uint4 v0, v1;
    if (HAS_V) {
      v0 = lds128(src + 1024);
      v1 = lds128(src + 1536);
    }
    issue(it + kStages - 1);

    // ---- partial dot products: 2 tokens x G heads over this lane's 8 dims ---------------------
    float vals[16];
    {
      const uint32_t kw[2][4] = {{k0.x, k0.y, k0.z, k0.w}, {k1.x, k1.y, k1.z, k1.w}};
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        u64 kp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) kp[i] = widen2(kw[t][i]);
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          if (h < G) {
            u64 s2 = fmul2(kp[0], q2[h][0]);
#pragma unroll
            for (int i = 1; i < 4; ++i) s2 = ffma2(kp[i], q2[h][i], s2);
            float lo, hi;
            unpack2(s2, lo, hi);
            vals[t * 8 + h] = lo + hi;
          } else {
            vals[t * 8 + h] = 0.f;
          }
        }
      }
    }
    // ---- reduce-scatter over the 16 lanes of a row: lane l16 ends with value index l16 --------
    float x;
    {
      const bool b3 = l16 & 8, b2 = l16 & 4, b1 = l16 & 2, b0 = l16 & 1;
      float v8[8], v4[4], v2[2];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float send = b3 ? vals[i] : vals[i + 8];
        const float keep = b3 ? vals[i + 8] : vals[i];
        v8[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float send = b2 ? v8[i] : v8[i + 4];
        const float keep = b2 ? v8[i + 4] : v8[i];
        v4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float send = b1 ? v4[i] : v4[i + 2];
        const float keep = b1 ? v4[i + 2] : v4[i];
        v2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
      }
      const float send = b0 ? v2[0] : v2[1];
      const float keep = b0 ? v2[1] : v2[0];
      x = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    // ---- owner lane: online softmax for (token, head) ----------------------------------------
    const int tok = (warp + it * kAttnWarps) * kQuad + half * 2 + own_tt;   // index inside the chunk
    const bool valid = own_head_ok && tok < cnt;
    x = valid ? x : -INFINITY;
    if (logit_row != nullptr && valid) {
      const int pos = start + tok;                     // dense / scoring mode: position == list index
      if (pos >= vis_lo && pos < vis_hi && pos - vis_lo < a.n_stride) logit_row[pos - vis_lo] = x;
    }
    float mx = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
    const bool raise = mx > m_ref + kRescaleSlack;
    if (__any_sync(0xffffffffu, raise)) {
      const float alpha = raise ? fast_exp2(m_ref - mx) : 1.f;     // m_ref = -inf gives 0
      if (raise) m_ref = mx;
      l_part *= alpha;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float ah = __shfl_sync(0xffffffffu, alpha, h);
        const u64 a2 = pack2(ah, ah);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc2[h][i] = fmul2(acc2[h][i], a2);
      }
    }
    const float p = valid ? fast_exp2(x - m_ref) : 0.f;
    l_part += p;

    if (HAS_V) {
      float* slot = prob_s + (it & 1) * 32;
      slot[lane] = p;
      __syncwarp();
      const float4* pv = reinterpret_cast<const float4*>(slot + half * 16);
      const float4 pa = pv[0], pb = pv[1], pc = pv[2], pd = pv[3];
      const float pp[2][8] = {{pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w},
                              {pc.x, pc.y, pc.z, pc.w, pd.x, pd.y, pd.z, pd.w}};
      const uint32_t vw[2][4] = {{v0.x, v0.y, v0.z, v0.w}, {v1.x, v1.y, v1.z, v1.w}};
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        u64 vp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) vp[i] = widen2(vw[t][i]);
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const u64 p2 = pack2(pp[t][h], pp[t][h]);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc2[h][i] = ffma2(vp[i], p2, acc2[h][i]);
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- merge inside the warp -----------------------------------------------------------------
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 8);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 16);
  float acc[G][8];
  if (HAS_V) {
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float lo, hi;
        unpack2(acc2[h][i], lo, hi);
        lo += __shfl_xor_sync(0xffffffffu, lo, 16);
        hi += __shfl_xor_sync(0xffffffffu, hi, 16);
        acc[h][2 * i] = lo;
        acc[h][2 * i + 1] = hi;
      }
  }
  __syncthreads();                                     // every warp is done with its ring

  // ---- merge across warps (re-using the ring space) and emit the split's partial --------------
  float* m_s = reinterpret_cast<float*>(smem + L::ring);            // [warps][8]
  float* l_s = m_s + kAttnWarps * 8;                                 // [warps][8]
  float* acc_s = l_s + kAttnWarps * 8;                               // [warps][G][128]
  if (lane < 8) {
    m_s[warp * 8 + lane] = (lane < G) ? m_ref : -INFINITY;
    l_s[warp * 8 + lane] = (lane < G) ? l_part : 0.f;
  }
  if (HAS_V && half == 0) {
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float4* dst = reinterpret_cast<float4*>(acc_s + (warp * G + h) * kHeadDim + l16 * 8);
      dst[0] = make_float4(acc[h][0], acc[h][1], acc[h][2], acc[h][3]);
      dst[1] = make_float4(acc[h][4], acc[h][5], acc[h][6], acc[h][7]);
    }
  }
  __syncthreads();
  const int64_t item = (static_cast<int64_t>(b) * a.num_kv_heads + g) * a.max_chunks + c;
  for (int o = tid; o < G * kHeadDim; o += kThreads) {
    const int h = o / kHeadDim, dd = o % kHeadDim;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, m_s[w * 8 + h]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float mw = m_s[w * 8 + h];
      const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
      den += l_s[w * 8 + h] * sc;
      if (HAS_V) num += acc_s[(w * G + h) * kHeadDim + dd] * sc;
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
