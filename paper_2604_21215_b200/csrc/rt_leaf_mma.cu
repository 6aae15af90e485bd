// Leaf recurrence kernel, bf16 / tiled-schedule version: the sequential part of Algorithm 1
// for the positions [t0, t1) of one leaf, all B <= 16 sequences at once.
//
// Same decomposition as the generic leaf kernel (one persistent CTA per SM, each CTA owning a
// fixed slice of the output rows of W_o, W_up, W_down, W_k, W_v in shared memory), but built
// for latency, because a token step is a chain of five all-to-all exchanges of small vectors:
//   * exchange words carry their own validity flag.  Every published 64-bit word holds a
//     payload (two bf16, or one fp32) and the 32-bit sequence number of the token step.
//     A consumer polls the payload words themselves: one L2 round trip per exchange, no
//     separate fence + counter + reload.  Flags are unique per step of an API call and the
//     buffers are zeroed at the start of the call.
//   * the mat-vec products run on the tensor cores as m16n8k16 MMAs with the sequences as
//     the M dimension (rows without a sequence are zero) and 8 weight rows as the N dimension,
//     K split over the MMA warps of a group and reduced through shared memory.  The fragments
//     of the activations are exactly the polled words; weight fragments are 8-byte shared loads.
//   * sequences are independent (Sec. 2.2 states the layer per sequence), and a token step is
//     bound by the latency of its exchanges, not by throughput.  The batch is therefore split
//     into NG groups of sequences, each with its own MMA warps, exchange buffers, flags and
//     counters, all reading the same weights in shared memory: while one group's words are in
//     flight the other groups' products run.
//   * two extra warps per CTA do the in-leaf attention (Algorithm 2 with one key at a time):
//     each owns one (sequence, head) pair and keeps the running stats (m, l, o) of every query
//     of the leaf in shared memory.  When the pair (k_j, v_j) arrives it first finishes query
//     j+1 (the only one on the critical path) and publishes c_{j+1} = o/l, and only then folds
//     the new pair into the later queries of the leaf, while the rest of the chip is busy with
//     the mat-vecs of step j+1.  These warps also apply qkRMS to k_j and write the caches.
#include <cuda_bf16.h>

#include <type_traits>

#include "rt_kernels.h"

namespace rt {

constexpr int kAttnSlots = 2;
constexpr int kNT = 4;                  // n-tiles (8 weight rows each) per pass
constexpr int kSlots = 8;               // sequence slots of a group: the MMA rows that carry data
constexpr int kRanges = kLeafMmaRanges; // completion counters of a group's g vector (ranges of d_ff)
constexpr int kQStride = kHeadDim + 2;  // bf16 elements per query row in shared memory
constexpr int kOStride = kHeadDim + 1;  // floats per o row in shared memory

struct LeafMmaLayout {
  int max_nd, max_nf;          // weight rows per CTA (upper bounds): d-row matrices, W_up
  int stride_d, stride_f;      // shared-memory row strides in elements (K + 16)
  int lf;                      // leaf capacity of the attention state
  int ng, wg;                  // sequence groups, MMA warps per group
  size_t off_grp, grp_bytes;   // per-group scratch: abort word, red[2], ssq[2], own rows of h
  size_t g_red, g_ssq, g_hown; // offsets inside a group's scratch
  size_t off_wo, off_wup, off_wdn, off_wk, off_wv, off_attn, attn_bytes, total;
};

LeafMmaLayout leaf_mma_layout(int d, int dff, int grid, int lf, int slots, int ng, int wg) {
  LeafMmaLayout L;
  L.max_nd = 2 * ceil_div(d / 2, grid);
  L.max_nf = 2 * ceil_div(dff / 2, grid);
  L.stride_d = d + 16;
  L.stride_f = dff + 16;
  L.lf = lf;
  L.ng = ng; L.wg = wg;
  size_t g = 16;                                              // the group's two abort words (used alternately)
  L.g_red = g;   g += 2 * sizeof(float2) * wg * kNT * 32;     // two buffers, used alternately
  L.g_ssq = g;   g += 2 * sizeof(float) * wg * kSlots;
  L.g_hown = g;  g += align_up(sizeof(float) * kSlots * (size_t)L.max_nd, 16);
  L.grp_bytes = align_up(g, 16);
  size_t o = 0;
  L.off_grp = o;   o += L.grp_bytes * ng;
  L.attn_bytes = align_up((size_t)lf * kQStride * 2 + (size_t)lf * kOStride * 4 + (size_t)lf * 8 + 2 * kHeadDim * 4, 16);
  L.off_attn = o;  o += L.attn_bytes * slots;
  o = align_up(o, 128);
  L.off_wo = o;    o += (size_t)L.max_nd * L.stride_d * 2;
  L.off_wup = o;   o += (size_t)L.max_nf * L.stride_d * 2;
  L.off_wdn = o;   o += (size_t)L.max_nd * L.stride_f * 2;
  L.off_wk = o;    o += (size_t)L.max_nd * L.stride_d * 2;
  L.off_wv = o;    o += (size_t)L.max_nd * L.stride_d * 2;
  L.total = o;
  return L;
}

// ---- small device helpers -------------------------------------------------------------------
__device__ __forceinline__ float gelu_erf_f(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)); }
__device__ __forceinline__ float bf_lo(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(unsigned u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ unsigned pack_bf2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const unsigned*>(&v);
}
// Every published word is one 64-bit scalar (payload in the low half, step number in the high
// half), so a reader never sees a payload without its flag.  Loads fetch two adjacent words.
__device__ __forceinline__ uint4 ld_relaxed_v4(const void* p) {
  unsigned long long w0, w1;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
  return make_uint4((unsigned)w0, (unsigned)(w0 >> 32), (unsigned)w1, (unsigned)(w1 >> 32));
}
// The same load under a predicate (no branch): when `on` is zero nothing is read and the result is
// two zero words (flag 0 never matches a step number).
__device__ __forceinline__ uint4 ld_relaxed_v4_if(const void* p, unsigned on) {
  unsigned long long w0 = 0ull, w1 = 0ull;
  asm volatile("{\n .reg .pred q;\n setp.ne.u32 q, %3, 0;\n @q ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];\n}"
               : "+l"(w0), "+l"(w1) : "l"(p), "r"(on) : "memory");
  return make_uint4((unsigned)w0, (unsigned)(w0 >> 32), (unsigned)w1, (unsigned)(w1 >> 32));
}
// 8 bytes through L2 under a predicate (zeros when `on` is zero).  An asm statement, so that a run
// of these stays a run of loads: written as plain loads the compiler placed each one's first use
// right behind it and the round trips added up.
__device__ __forceinline__ uint2 ld_cg_v2_if(const void* p, unsigned on) {
  uint2 w = make_uint2(0u, 0u);
  asm volatile("{\n .reg .pred q;\n setp.ne.u32 q, %3, 0;\n @q ld.global.cg.v2.u32 {%0,%1}, [%2];\n}"
               : "+r"(w.x), "+r"(w.y) : "l"(p), "r"(on) : "memory");
  return w;
}
__device__ __forceinline__ void st_relaxed_u64(void* p, unsigned lo, unsigned hi) {
  const unsigned long long w = ((unsigned long long)hi << 32) | lo;
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(w) : "memory");
}
__device__ __forceinline__ void st_relaxed_v4(void* p, unsigned a, unsigned b, unsigned c, unsigned d) {
  const unsigned long long w0 = ((unsigned long long)b << 32) | a, w1 = ((unsigned long long)d << 32) | c;
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1,%2};" ::"l"(p), "l"(w0), "l"(w1) : "memory");
}
// m16n8k16 with rows 8..15 of A all zero: the sequences of a group fill rows 0..7 only, so c[2] and c[3]
// (rows 8..15 of the result) stay zero and only c[0], c[1] are used.
__device__ __forceinline__ void mma_bf16_top(float (&c)[4], unsigned a0, unsigned a2, unsigned b0, unsigned b1) {
  const unsigned zero = 0u;
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}
// Barrier over the MMA warps of one group (named barrier 1 + group).
template <int WG>
__device__ __forceinline__ void group_sync(int grp) {
  asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(WG * 32) : "memory");
}

// A wait that ran out: record it for the host and tell every other waiter to leave.
__device__ __noinline__ void report_timeout(SyncArea* s) {
  s->status = RT_ERR_TIMEOUT;
  __threadfence();
  atomicExch(&s->abort_flag, 1u);
}
// Called every few polls: true when the wait must be abandoned.
__device__ __forceinline__ bool wait_expired(SyncArea* s, unsigned long long& t_start) {
  if (*reinterpret_cast<volatile unsigned*>(&s->abort_flag)) return true;
  const unsigned long long now = globaltimer_ns();
  if (t_start == 0) { t_start = now; return false; }
  if (now - t_start > kWaitLimitNs) { report_timeout(s); return true; }
  return false;
}

// Exchange words of a group's [sequences, K] bf16 vector are stored in the order the MMA fragments
// are read: [k-step of 16][8 sequence slots][4 groups of 4 k][2 words of 2 k], so that one warp-wide
// 16-byte load (8 sequences x 4 groups) covers 512 contiguous bytes.  Index of the word that holds
// elements k, k+1 (k even) of the group's sequence b:
__device__ __forceinline__ size_t ll_word(int b, int k) {
  return ((size_t)((k >> 4) * kSlots + b) * 4 + ((k & 15) >> 2)) * 2 + ((k & 3) >> 1);
}
constexpr int kWordsPerKStep = kSlots * 8;      // 64-bit words of one k-step
// g as packed bf16 in the order the fragments are read: [k-step of 16][8 sequence slots][16 k], so
// the 8 sequences x 32 bytes one warp-wide load touches are 256 contiguous bytes
__device__ __forceinline__ size_t g_index(int b, int k) { return ((size_t)((k >> 4) * kSlots + b) << 4) + (size_t)(k & 15); }
constexpr int kGElemsPerKStep = kSlots * 16;

// Sum of squares (of the raw values) and optional gain for one k-step of fragments; gp points
// at this thread's 4 gains of the k-step (or is null).
__device__ __forceinline__ void frag_ssq_gain(unsigned& a0, unsigned& a2, const __nv_bfloat16* gp, float& sq) {
  const float v0 = bf_lo(a0), v1 = bf_hi(a0), v2 = bf_lo(a2), v3 = bf_hi(a2);
  sq += v0 * v0 + v1 * v1 + v2 * v2 + v3 * v3;
  if (gp) {
    const uint2 gw = *reinterpret_cast<const uint2*>(gp);
    a0 = pack_bf2(v0 * bf_lo(gw.x), v1 * bf_hi(gw.x));
    a2 = pack_bf2(v2 * bf_lo(gw.y), v3 * bf_hi(gw.y));
  }
}

// ---- attention warp: one (sequence, head) pair for the whole leaf ----------------------------
template <bool TIMERS>
__device__ void attention_role(const LeafParams& p, const LeafMmaLayout& L, unsigned char* smem_slot, int pair,
                               const unsigned long long* ll_kv, unsigned long long* ll_c_all, size_t grp_words_d) {
  const int lane = threadIdx.x & 31;
  const int B = p.B, d = p.d, H = p.H;
  const int b = pair / H, h = pair % H;
  const int Bg = (B + L.ng - 1) / L.ng;
  const int grp = b / Bg, bl = b - grp * Bg;                    // the sequence's group and its slot there
  unsigned long long* ll_c = ll_c_all + (size_t)grp * grp_words_d;
  const int n = p.t1 - p.t0;
  __nv_bfloat16* qs = reinterpret_cast<__nv_bfloat16*>(smem_slot);
  float* os = reinterpret_cast<float*>(smem_slot + (size_t)L.lf * kQStride * 2);
  float* ms = os + (size_t)L.lf * kOStride;
  float* ls = ms + L.lf;
  float* kbuf = ls + L.lf;
  float* vbuf = kbuf + kHeadDim;
  const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(p.q);
  const __nv_bfloat16* g_k = reinterpret_cast<const __nv_bfloat16*>(p.g_k);
  __nv_bfloat16* kc = reinterpret_cast<__nv_bfloat16*>(p.k_cache);
  __nv_bfloat16* vc = reinterpret_cast<__nv_bfloat16*>(p.v_cache);
  const bool qkn = (p.norm_flags & RT_NORM_QK) != 0;
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;     // ALiBi distances, in log2 units

  // queries and carried stats of the leaf (written by earlier kernels of this call)
  for (int i = 0; i < n; ++i) {
    const size_t row = (size_t)(p.t0 + i) * B + b;
    *reinterpret_cast<unsigned*>(qs + i * kQStride + 2 * lane) =
        *reinterpret_cast<const unsigned*>(q + row * d + h * kHeadDim + 2 * lane);
    os[i * kOStride + lane] = p.st_o[row * d + h * kHeadDim + lane];
    os[i * kOStride + lane + 32] = p.st_o[row * d + h * kHeadDim + lane + 32];
  }
  for (int i = lane; i < n; i += 32) {
    const size_t row = (size_t)(p.t0 + i) * B + b;
    ms[i] = p.st_m[row * H + h];
    ls[i] = p.st_l[row * H + h];
  }
  __syncwarp();
  const float gk0 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane) : 1.0f;
  const float gk1 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane + 1) : 1.0f;
  unsigned long long* c_word = ll_c + ll_word(bl, h * kHeadDim + 2 * lane);
  // c of the first position: nothing of this leaf to fold in
  {
    const float il = 1.0f / ls[0];
    st_relaxed_u64(c_word, pack_bf2(os[2 * lane] * il, os[2 * lane + 1] * il), p.seq_base + 1u);
  }
  const unsigned long long* k_words = ll_kv + (size_t)b * (2 * d) + h * kHeadDim + 2 * lane;
  const unsigned long long* v_words = k_words + d;
  const bool timing = TIMERS && (pair == 0 && lane == 0);
  unsigned long long a_work = 0, a_wait = 0, t_mark = timing ? globaltimer_ns() : 0ull;
  for (int j = 0; j < n; ++j) {
    const unsigned seq = p.seq_base + (unsigned)j + 1u;      // step that reveals position t0 + j
    uint4 kw, vw;
    if (timing) { const unsigned long long now = globaltimer_ns(); a_work += now - t_mark; t_mark = now; }
    unsigned spins = 0;
    unsigned long long t_start = 0;
    while (true) {
      kw = ld_relaxed_v4(k_words);
      vw = ld_relaxed_v4(v_words);
      const bool ok = kw.y == seq && kw.w == seq && vw.y == seq && vw.w == seq;
      if (__all_sync(0xffffffffu, ok)) break;
      if ((++spins & 63u) == 0u) {
        int bad = 0;
        if (lane == 0) bad = wait_expired(p.sync, t_start) ? 1 : 0;
        if (__shfl_sync(0xffffffffu, bad, 0)) return;
      }
    }
    if (timing) { const unsigned long long now = globaltimer_ns(); a_wait += now - t_mark; t_mark = now; }
    // Eq. (1): qkRMS over the head, then the storage rounding the cache applies
    const float k0 = __uint_as_float(kw.x), k1 = __uint_as_float(kw.z);
    const float ss = warp_sum(k0 * k0 + k1 * k1);
    const float rs = qkn ? rsqrtf(ss * (1.0f / kHeadDim) + p.eps) : 1.0f;
    const unsigned kq = pack_bf2(k0 * rs * gk0, k1 * rs * gk1);
    const unsigned vq = pack_bf2(__uint_as_float(vw.x), __uint_as_float(vw.z));
    const size_t crow = ((size_t)(p.t0 + j) * B + b) * d + h * kHeadDim + 2 * lane;
    *reinterpret_cast<unsigned*>(kc + crow) = kq;
    *reinterpret_cast<unsigned*>(vc + crow) = vq;
    if (j + 1 >= n) break;
    const float kf0 = bf_lo(kq), kf1 = bf_hi(kq), vf0 = bf_lo(vq), vf1 = bf_hi(vq);
    {
      // critical path: finish query j+1 and publish c_{j+1}
      const int i = j + 1;
      const unsigned qw = *reinterpret_cast<const unsigned*>(qs + i * kQStride + 2 * lane);
      const float s = warp_sum(bf_lo(qw) * kf0 + bf_hi(qw) * kf1) * p.scale_log2 - slope_l2;      // distance (j+1) - j = 1
      const float m_old = ms[i], l_old = ls[i];
      const float m_new = fmaxf(m_old, s);
      const float corr = exp2f(m_old - m_new), pj = exp2f(s - m_new);
      const float il = 1.0f / (l_old * corr + pj);
      const float o0 = os[i * kOStride + 2 * lane] * corr + pj * vf0;
      const float o1 = os[i * kOStride + 2 * lane + 1] * corr + pj * vf1;
      st_relaxed_u64(c_word, pack_bf2(o0 * il, o1 * il), seq + 1u);
    }
    // off the critical path: fold (k_j, v_j) into the later queries of the leaf, one query per lane
    kbuf[2 * lane] = kf0; kbuf[2 * lane + 1] = kf1;
    vbuf[2 * lane] = vf0; vbuf[2 * lane + 1] = vf1;
    __syncwarp();
    for (int i = j + 2 + lane; i < n; i += 32) {
      const __nv_bfloat16* qi = qs + i * kQStride;
      float s = 0.f;
#pragma unroll 8
      for (int e = 0; e < kHeadDim; e += 2) {
        const unsigned qw = *reinterpret_cast<const unsigned*>(qi + e);
        s += bf_lo(qw) * kbuf[e] + bf_hi(qw) * kbuf[e + 1];
      }
      s = s * p.scale_log2 - slope_l2 * (float)(i - j);
      const float m_old = ms[i];
      const float m_new = fmaxf(m_old, s);
      const float corr = exp2f(m_old - m_new), pj = exp2f(s - m_new);
      ms[i] = m_new;
      ls[i] = ls[i] * corr + pj;
      float* oi = os + i * kOStride;
#pragma unroll 8
      for (int e = 0; e < kHeadDim; ++e) oi[e] = oi[e] * corr + pj * vbuf[e];
    }
    __syncwarp();
  }
  if (timing) { atomicAdd(&p.sync->phase_ns[0], a_work); atomicAdd(&p.sync->phase_ns[1], a_wait); }
}

// NG groups of WG MMA warps.  TIMERS and GAINS are compile-time: the token step is a latency chain of code that runs
// once per token, and every instruction and live register that is compiled in costs time even when its branch is not
// taken.
template <int NG, int WG, bool TIMERS, bool GAINS>
__global__ void __launch_bounds__((NG * WG + kAttnSlots) * 32, 1) leaf_mma_kernel(const LeafParams p, const LeafMmaLayout L,
                                                                                  const LeafMmaBuffers buf) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int kThreads = (NG * WG + kAttnSlots) * 32;
  // k-steps per round of polled loads / of loads of g (W_down): as many as the registers of the launch shape
  // hold (the register file is dealt out per 4 warps: up to 12 warps leave a thread 168 registers, 20 leave 96)
  constexpr int KC = NG * WG > 8 ? 8 : (WG >= 8 ? 8 : 16);
  constexpr int KD = NG * WG > 8 ? 16 : 32;
  constexpr int RPW = kRanges / WG;                              // completion counters a warp waits for
  static_assert(kRanges % WG == 0 && RPW >= 1, "ranges of g are dealt out evenly to the warps of a group");
  __nv_bfloat16* s_wo = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wo);
  __nv_bfloat16* s_wup = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wup);
  __nv_bfloat16* s_wdn = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wdn);
  __nv_bfloat16* s_wk = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wk);
  __nv_bfloat16* s_wv = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wv);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int B = p.B, d = p.d, dff = p.dff;
  if (*reinterpret_cast<volatile unsigned*>(&p.sync->abort_flag)) return;
  // rows are dealt out in pairs so that a published word (two consecutive rows) has one owner
  const int d_lo = 2 * (int)((long long)(d / 2) * cta / G), d_hi = 2 * (int)((long long)(d / 2) * (cta + 1) / G);
  const int f_lo = 2 * (int)((long long)(dff / 2) * cta / G), f_hi = 2 * (int)((long long)(dff / 2) * (cta + 1) / G);
  const int nd = d_hi - d_lo, nf = f_hi - f_lo;

  if (tid < 2 * NG) reinterpret_cast<volatile int*>(smem + L.off_grp + (size_t)(tid >> 1) * L.grp_bytes)[tid & 1] = 0;
  {
    auto stage = [&](__nv_bfloat16* dst, int dst_stride, const void* src_base, int row_lo, int nrows, int K) {
      const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(src_base) + (size_t)row_lo * K);
      const int per_row = K / 8;
      for (int i = tid; i < nrows * per_row; i += kThreads) {
        const int r = i / per_row, v = i % per_row;
        *reinterpret_cast<uint4*>(dst + (size_t)r * dst_stride + v * 8) = src[(size_t)r * per_row + v];
      }
    };
    stage(s_wo, L.stride_d, p.w_o, d_lo, nd, d);
    stage(s_wup, L.stride_d, p.w_up, f_lo, nf, d);
    stage(s_wdn, L.stride_f, p.w_down, d_lo, nd, dff);
    stage(s_wk, L.stride_d, p.w_k, d_lo, nd, d);
    stage(s_wv, L.stride_d, p.w_v, d_lo, nd, d);
  }
  __syncthreads();

  if (warp >= NG * WG) {
    const int slot = warp - NG * WG;
    const int pair = cta + slot * G;
    if (pair < B * p.H)
      attention_role<TIMERS>(p, L, smem + L.off_attn + (size_t)slot * L.attn_bytes, pair, buf.ll_kv, buf.ll_c, buf.grp_words_d);
    return;
  }

  // ------------------------------ MMA warps ------------------------------
  // The four mat-vec phases of a token step run through ONE inlined copy of the code below (a loop
  // over the phase index): the step executes once per token, so four straight-line copies would
  // only thrash the instruction cache, and calls through a real function would put the fragments
  // and accumulators on the stack, where every access is an L2 round trip.
  const int grp = NG > 1 ? warp / WG : 0, lw = NG > 1 ? warp % WG : warp;
  const int Bg = (B + NG - 1) / NG;
  const int b_lo = grp * Bg;
  const int nb = B - b_lo < Bg ? B - b_lo : Bg;                  // sequences of this group
  if (nb <= 0) return;                                           // (the launcher never makes an empty group)
  unsigned char* gs = smem + L.off_grp + (size_t)grp * L.grp_bytes;
  // A warp whose wait ran out sets the abort word of the pass it is in; every warp of the group reads that word
  // right after the pass's barrier, so all of them leave at the same barrier (two words, alternating like the
  // reduction buffers: a warp already in the next pass cannot disturb a slower warp's read of this one)
  volatile int* s_abort = reinterpret_cast<volatile int*>(gs);
  float2* red = reinterpret_cast<float2*>(gs + L.g_red);
  float* ssq_red = reinterpret_cast<float*>(gs + L.g_ssq);
  float* hown = reinterpret_cast<float*>(gs + L.g_hown);
  unsigned long long* ll_c = buf.ll_c + (size_t)grp * buf.grp_words_d;
  unsigned long long* ll_h = buf.ll_h + (size_t)grp * buf.grp_words_d;
  unsigned long long* ll_z = buf.ll_z + (size_t)grp * buf.grp_words_d;
  __nv_bfloat16* g_pk = reinterpret_cast<__nv_bfloat16*>(buf.ll_g + (size_t)grp * buf.grp_words_g);
  unsigned* g_cnt = buf.g_cnt + (size_t)grp * kRanges * 32;      // one 128-byte line per counter
  unsigned long long* ll_kv = buf.ll_kv;

  const int g = lane >> 2, c = lane & 3;
  const bool pre = (p.norm_flags & RT_NORM_PRE) != 0;
  const bool kv_norm = pre && !(p.norm_flags & RT_NORM_SKIP_Z);
  const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(p.x);
  __nv_bfloat16* z = reinterpret_cast<__nv_bfloat16*>(p.z);
  const float inv_d = 1.0f / (float)d;
  const int nt_d = (nd + 7) / 8, nt_f = (nf + 7) / 8;
  const bool has0 = g < nb;
  const int bq = b_lo + (has0 ? g : 0);                          // this lane's sequence in the batch
  const int g0 = has0 ? g : 0;                                   // slot read by lanes without a sequence (masked)
  const unsigned keep0 = has0 ? 0xffffffffu : 0u;
  const bool timing = TIMERS && (cta == 0 && tid == 0);
  unsigned long long t_ph = timing ? globaltimer_ns() : 0ull;

  // Completion counters of g: the k-steps of d_ff are cut into kRanges ranges, warp lw multiplies the RPW ranges
  // [lw * RPW, (lw + 1) * RPW).  A producer CTA bumps the counter of every range its rows of W_up fall in once per
  // token step, so a consumer warp waits for the few CTAs that write its part of g, not for the whole grid.
  const int n_ks_f = dff / 16;
  const int ks_per_range = (n_ks_f + kRanges - 1) / kRanges;
  const int my_r_lo = nf > 0 ? (f_lo / 16) / ks_per_range : 0;   // ranges this CTA produces for
  const int my_r_hi = nf > 0 ? ((f_hi - 1) / 16) / ks_per_range : -1;
  unsigned cnt_per_step = 0;                                     // lane i < RPW: arrivals per step at range lw*RPW + i
  if (lane < RPW) {
    const int r = lw * RPW + lane;
    for (int cc = 0; cc < G; ++cc) {
      const int lo = 2 * (int)((long long)(dff / 2) * cc / G), hi = 2 * (int)((long long)(dff / 2) * (cc + 1) / G);
      if (hi > lo && (lo / 16) / ks_per_range <= r && ((hi - 1) / 16) / ks_per_range >= r) ++cnt_per_step;
    }
  }
  unsigned pass = 0;                                             // passes so far: selects the reduction buffer

  for (int t = p.t0; t < p.t1; ++t) {
    const unsigned seq = p.seq_base + (unsigned)(t - p.t0) + 1u;
#pragma unroll 1
    for (int ph = 0; ph < 4; ++ph) {                              // 0: W_o   1: W_up   2: W_down   3: W_k | W_v
      // ---- what this phase multiplies ----
      const int K = (ph == 2) ? dff : d;
      const int stride = (ph == 2) ? L.stride_f : L.stride_d;
      const int nrows = (ph == 1) ? nf : nd;                       // rows per matrix of this phase
      const int nt_one = (ph == 1) ? nt_f : nt_d;
      const int nt_all = (ph == 3) ? 2 * nt_d : nt_one;
      const unsigned long long* act_ll = (ph == 0) ? ll_c : ((ph == 1) ? ll_h : ll_z);
      const __nv_bfloat16* gain = nullptr;
      bool want_ssq = false;
      if (ph == 1 && pre) { if (GAINS) gain = reinterpret_cast<const __nv_bfloat16*>(p.g_mlp); want_ssq = true; }
      if (ph == 3 && kv_norm) { if (GAINS) gain = reinterpret_cast<const __nv_bfloat16*>(p.g_kv); want_ssq = true; }
      const __nv_bfloat16* gp = (GAINS && gain) ? gain + 4 * c : nullptr;
      unsigned long long wait_ns = 0;
      bool alive = true;
      const int n_ks = K / 16;
      const int ks_per_warp = (ph == 2) ? ks_per_range * RPW : (n_ks + WG - 1) / WG;
      const int ks0 = lw * ks_per_warp < n_ks ? lw * ks_per_warp : n_ks;
      const int ks1 = ks0 + ks_per_warp < n_ks ? ks0 + ks_per_warp : n_ks;
      if (ph == 2) {
        // this warp's part of g (packed bf16, written by a few CTAs) must be complete before it multiplies by W_down
        const unsigned long long tb = timing ? globaltimer_ns() : 0ull;
        const unsigned target = seq * cnt_per_step;
        unsigned spins = 0;
        unsigned long long t_start = 0;
        while (true) {
          bool ok = true;
          if (lane < RPW) ok = ld_acquire_u32(g_cnt + (size_t)(lw * RPW + lane) * 32) >= target;
          if (__all_sync(0xffffffffu, ok)) break;
          if ((++spins & 63u) == 0u) {
            int bad = 0;
            if (lane == 0) bad = wait_expired(p.sync, t_start) ? 1 : 0;
            if (__shfl_sync(0xffffffffu, bad, 0)) { s_abort[pass & 1u] = 1; alive = false; break; }
          }
        }
        if (timing) wait_ns += globaltimer_ns() - tb;
      }

      const int tile_step = (ph == 2) ? 1 : kNT;                   // W_down: one tile per pass (see below)
      for (int t0n = 0; t0n < nt_all; t0n += tile_step, ++pass) {
        const int n_tiles = nt_all - t0n < tile_step ? nt_all - t0n : tile_step;
        // this thread's 8 bytes of weight row g (clamped to the rows that exist) of each tile, at k = 4c
        const unsigned char* wp[kNT];
#pragma unroll
        for (int i = 0; i < kNT; ++i) {
          const int ti = t0n + i < nt_all ? t0n + i : t0n;
          const bool second = (ph == 3) && ti >= nt_d;             // W_v tiles follow the W_k tiles
          const int r0 = (second ? ti - nt_d : ti) * 8;
          const int valid = nrows - r0 < 8 ? nrows - r0 : 8;
          const int r = r0 + (g < valid ? g : valid - 1);
          const __nv_bfloat16* wbase = (ph == 0) ? s_wo : (ph == 1) ? s_wup : (ph == 2) ? s_wdn : (second ? s_wv : s_wk);
          wp[i] = reinterpret_cast<const unsigned char*>(wbase + (size_t)r * stride + 4 * c);
        }
        // rows this thread finishes after the reduction (warp w finishes tile t0n + w)
        const int ti_e = t0n + lw;
        const bool second_e = (ph == 3) && ti_e >= nt_d;
        const int rl = (second_e ? ti_e - nt_d : ti_e) * 8 + 2 * c;
        const bool mine = lw < n_tiles && rl < nrows && has0;
        unsigned xw0 = 0;
        if (ph == 0 && mine)                                       // x_t for the residual, fetched before the wait
          xw0 = *reinterpret_cast<const unsigned*>(x + (size_t)bq * p.x_bs + (size_t)t * p.x_ts + d_lo + rl);

        // The loops below are written without branches around the loads and the products (indices
        // are clamped, missing sequences and k-steps contribute zeros): a branch per product costs
        // more here than the product.
        float acc[kNT][4];
#pragma unroll
        for (int nt = 0; nt < kNT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
        float sq0 = 0.f;
        if (ph == 2) {
          // W_down reads g as packed bf16 behind its completion counters: plain loads, and a whole round of this
          // warp's k-steps is in flight before the first product.  One tile per pass; the four accumulators cut
          // the dependent chain of products.
          const __nv_bfloat16* b0p = g_pk + g_index(g0, 4 * c);          // + kGElemsPerKStep elements per k-step
          for (int kc0 = ks0; kc0 < ks1; kc0 += KD) {
            const int n_here = ks1 - kc0;
            uint2 w0[KD];
#pragma unroll
            for (int i = 0; i < KD; ++i)
              w0[i] = ld_cg_v2_if(b0p + (size_t)(kc0 + (i < n_here ? i : 0)) * kGElemsPerKStep, (i < n_here ? 1u : 0u) & keep0);
            const unsigned char* wd = wp[0] + (size_t)kc0 * 32;
#pragma unroll
            for (int i = 0; i < KD; ++i) {
              const uint2 bw = *reinterpret_cast<const uint2*>(wd + (i < n_here ? i : 0) * 32);
              mma_bf16_top(acc[i & 3], w0[i].x, w0[i].y, bw.x, bw.y);
            }
          }
          acc[0][0] += acc[1][0] + acc[2][0] + acc[3][0];
          acc[0][1] += acc[1][1] + acc[2][1] + acc[3][1];
        } else
        for (int kc0 = ks0; kc0 < ks1; kc0 += KC) {
          unsigned a0[KC], a2[KC];
#pragma unroll
          for (int i = 0; i < KC; ++i) { a0[i] = a2[i] = 0u; }
          const int n_here = ks1 - kc0;                             // k-steps of this round (the rest stay zero)
          {
            // flag-carrying words: a k-step is 8 words per sequence, this thread takes the 2 adjacent ones at 4c
            const unsigned long long* base0 = act_ll + ll_word(g0, 4 * c) + (size_t)kc0 * kWordsPerKStep;
            unsigned need0 = 0;
#pragma unroll
            for (int i = 0; i < KC; ++i) {
              if (i < n_here) need0 |= (1u << i) & keep0;
            }
            unsigned spins = 0;
            unsigned long long t_start = 0;
            const unsigned long long t_poll = timing ? globaltimer_ns() : 0ull;
            while (alive) {
              // every outstanding word of the round is loaded (under a predicate, not a branch) before
              // any flag is looked at, so the loads overlap
              uint4 w0[KC];
#pragma unroll
              for (int i = 0; i < KC; ++i) w0[i] = ld_relaxed_v4_if(base0 + (size_t)(i < n_here ? i : 0) * kWordsPerKStep, (need0 >> i) & 1u);
#pragma unroll
              for (int i = 0; i < KC; ++i) {
                const bool okw = (w0[i].y == seq) & (w0[i].w == seq) & ((need0 >> i) & 1u);
                a0[i] = okw ? w0[i].x : a0[i];
                a2[i] = okw ? w0[i].z : a2[i];
                need0 &= okw ? ~(1u << i) : 0xffffffffu;
              }
              if (__all_sync(0xffffffffu, need0 == 0u)) break;
              if ((++spins & 63u) == 0u) {
                int bad = 0;
                if (lane == 0) bad = wait_expired(p.sync, t_start) ? 1 : 0;
                if (__shfl_sync(0xffffffffu, bad, 0)) { s_abort[pass & 1u] = 1; alive = false; }
              }
            }
            if (timing) wait_ns += globaltimer_ns() - t_poll;
          }
          const __nv_bfloat16* gc = (GAINS && gp) ? gp + (size_t)kc0 * 16 : nullptr;
          if (want_ssq) {
#pragma unroll
            for (int i = 0; i < KC; ++i) frag_ssq_gain(a0[i], a2[i], (GAINS && gc) ? gc + (i < n_here ? i : 0) * 16 : nullptr, sq0);
          }
          // products, specialised on the number of tiles so that none sits behind a branch
          auto products = [&](auto ntc) {
            constexpr int NTC = decltype(ntc)::value;
#pragma unroll
            for (int i = 0; i < KC; ++i) {
              const int off = ((i < n_here ? i : 0) + kc0) * 32;
#pragma unroll
              for (int nt = 0; nt < NTC; ++nt) {
                const uint2 bw = *reinterpret_cast<const uint2*>(wp[nt] + off);
                mma_bf16_top(acc[nt], a0[i], a2[i], bw.x, bw.y);
              }
            }
          };
          switch (n_tiles) {
            case 1: products(std::integral_constant<int, 1>{}); break;
            case 2: products(std::integral_constant<int, 2>{}); break;
            case 3: products(std::integral_constant<int, 3>{}); break;
            default: products(std::integral_constant<int, 4>{}); break;
          }
        }
        // ---- reduce the K split over the group's warps; warp w then holds the sums of tile t0n + w.  The buffers
        // alternate between passes, so one barrier per pass is enough: a warp can only write a buffer again after
        // it has passed the next pass's barrier, which every warp reaches after its reads of this pass ----
        if (!alive) s_abort[pass & 1u] = 1;
        float2* redb = red + (size_t)(pass & 1u) * (WG * kNT * 32);
        float* ssqb = ssq_red + (size_t)(pass & 1u) * (WG * kSlots);
#pragma unroll
        for (int nt = 0; nt < kNT; ++nt)
          if (nt < n_tiles) redb[(lw * kNT + nt) * 32 + lane] = make_float2(acc[nt][0], acc[nt][1]);
        if (want_ssq) {
          sq0 += __shfl_xor_sync(0xffffffffu, sq0, 1); sq0 += __shfl_xor_sync(0xffffffffu, sq0, 2);
          if (c == 0) ssqb[lw * kSlots + g] = sq0;
        }
        group_sync<WG>(grp);
        if (s_abort[pass & 1u]) return;
        // ---- epilogue: y0, y1 = rows rl, rl+1 of the tile this warp finishes, for the sequence of slot g ----
        if (lw < n_tiles) {
          float y0 = 0.f, y1 = 0.f, ssq = 0.f;
#pragma unroll
          for (int w = 0; w < WG; ++w) {
            const float2 v = redb[(w * kNT + lw) * 32 + lane];
            y0 += v.x; y1 += v.y;
          }
          if (want_ssq) {
#pragma unroll
            for (int w = 0; w < WG; ++w) ssq += ssqb[w * kSlots + g];
          }
          if (mine) {
            if (ph == 0) {                                            // h = x_t + alpha W_o c_t
              const float h0 = bf_lo(xw0) + p.alpha * y0, h1 = bf_hi(xw0) + p.alpha * y1;
              hown[g * L.max_nd + rl] = h0; hown[g * L.max_nd + rl + 1] = h1;
              st_relaxed_u64(ll_h + ll_word(g, d_lo + rl), pack_bf2(h0, h1), seq);
            } else if (ph == 1) {                                     // g = GELU(W_up RMS(h)), packed bf16
              const float rs = pre ? rsqrtf(ssq * inv_d + p.eps) : 1.0f;
              *reinterpret_cast<unsigned*>(g_pk + g_index(g, f_lo + rl)) = pack_bf2(gelu_erf_f(y0 * rs), gelu_erf_f(y1 * rs));
            } else if (ph == 2) {                                     // z_t = h + alpha W_down g   (layer output)
              const unsigned zw = pack_bf2(hown[g * L.max_nd + rl] + p.alpha * y0, hown[g * L.max_nd + rl + 1] + p.alpha * y1);
              *reinterpret_cast<unsigned*>(z + (size_t)bq * p.z_bs + (size_t)t * p.z_ts + d_lo + rl) = zw;
              st_relaxed_u64(ll_z + ll_word(g, d_lo + rl), zw, seq);
            } else {                                                  // raw k_t, v_t from RMS(z_t): Eqs. (1)-(2) before qkRMS
              const size_t col = (size_t)(second_e ? d : 0) + d_lo + rl;
              const float rs = kv_norm ? rsqrtf(ssq * inv_d + p.eps) : 1.0f;
              st_relaxed_v4(ll_kv + (size_t)bq * (2 * d) + col, __float_as_uint(y0 * rs), seq, __float_as_uint(y1 * rs), seq);
            }
          }
        }
      }
      if (ph == 1) {
        // all of this CTA's rows of g are written: tell the warps (of every CTA) that multiply those ranges.  The
        // release is cumulative over what the group barrier ordered before it.
        group_sync<WG>(grp);
        if (lw == 0 && lane <= my_r_hi - my_r_lo) red_release_add_u32(g_cnt + (size_t)(my_r_lo + lane) * 32, 1u);
      }
      if (timing) {
        const unsigned long long now = globaltimer_ns();
        atomicAdd(&p.sync->phase_ns[2 + 2 * ph], now - t_ph - wait_ns);        // fire-and-forget, no stack array
        atomicAdd(&p.sync->phase_ns[3 + 2 * ph], wait_ns);
        t_ph = now;
      }
    }
  }
}

// ------------------------------------------------------------------------------------ host

// Exchange-buffer sizes in 64-bit words (see LeafMmaBuffers): one group's c / h / z vector, one group's g vector.
size_t leaf_mma_words_d(int d) { return (size_t)(d / 16) * kWordsPerKStep; }
size_t leaf_mma_words_g(int dff) { return (size_t)(dff / 16) * kGElemsPerKStep / 4; }

// Picks the number of sequence groups, the leaf capacity and the launch shape; returns false when this kernel
// does not take the shape (the generic leaf kernel does).
bool leaf_mma_plan(int B, int d, int H, int dff, int want_leaf, int want_groups, LeafMmaLaunch* out) {
  int dev = 0, sms = 0, max_smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
  if (B > 16 || (d % 64) || (dff % 16) || B * H > kAttnSlots * sms) return false;
  // groups: as many as requested (or two), lowered until no group is empty and raised until none has more than 8 sequences
  int ng = want_groups > 0 ? want_groups : 2;
  if (ng != 1 && ng != 2 && ng != 4) return false;
  while (ng > 1 && (ng > B || ceil_div(B, ng) * (ng - 1) >= B)) ng /= 2;
  while (ng < kLeafMmaMaxGroups && ceil_div(B, ng) > kSlots) ng *= 2;
  if (ceil_div(B, ng) > kSlots) return false;
  const int wg = ng == 1 ? 8 : 4;
  const int cands[3] = {64, 32, 16};
  for (int lf : cands) {
    if (want_leaf && lf != want_leaf) continue;
    const LeafMmaLayout L = leaf_mma_layout(d, dff, sms, lf, ceil_div(B * H, sms), ng, wg);
    if (L.total <= (size_t)max_smem) {
      out->grid = sms; out->block = (ng * wg + kAttnSlots) * 32; out->smem = L.total; out->leaf = lf;
      out->groups = ng; out->warps_per_group = wg;
      return true;
    }
  }
  return false;
}

cudaError_t leaf_mma_launch(const LeafParams& p, const LeafMmaLaunch& l, const LeafMmaBuffers& buf, cudaStream_t s) {
  LeafMmaLayout L = leaf_mma_layout(p.d, p.dff, l.grid, l.leaf, ceil_div(p.B * p.H, l.grid), l.groups, l.warps_per_group);
  // compile-time variants: groups x warps per group, per-phase timers, RMS gains present
  const bool gains = p.g_mlp != nullptr || p.g_kv != nullptr;
  auto pick = [&](auto ng, auto wg) -> const void* {
    constexpr int NG = decltype(ng)::value, WG = decltype(wg)::value;
    if (p.timers) return gains ? reinterpret_cast<const void*>(&leaf_mma_kernel<NG, WG, true, true>)
                               : reinterpret_cast<const void*>(&leaf_mma_kernel<NG, WG, true, false>);
    return gains ? reinterpret_cast<const void*>(&leaf_mma_kernel<NG, WG, false, true>)
                 : reinterpret_cast<const void*>(&leaf_mma_kernel<NG, WG, false, false>);
  };
  const void* fn = nullptr;
  if (l.groups == 1 && l.warps_per_group == 8) fn = pick(std::integral_constant<int, 1>{}, std::integral_constant<int, 8>{});
  else if (l.groups == 2 && l.warps_per_group == 4) fn = pick(std::integral_constant<int, 2>{}, std::integral_constant<int, 4>{});
  else if (l.groups == 4 && l.warps_per_group == 4) fn = pick(std::integral_constant<int, 4>{}, std::integral_constant<int, 4>{});
  if (!fn) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.smem);
  if (e != cudaSuccess) return e;
  LeafParams pp = p;
  LeafMmaBuffers b = buf;
  void* args[] = {(void*)&pp, (void*)&L, (void*)&b};
  return cudaLaunchCooperativeKernel(fn, dim3(l.grid), dim3(l.block), args, l.smem, s);
}

}  // namespace rt
