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
//   * the mat-vec products run on the tensor cores as m16n8k16 MMAs with the B sequences as
//     the M dimension (rows >= B are zero) and 8 weight rows as the N dimension, K split over
//     the 8 MMA warps of the CTA and reduced through shared memory.  The fragments of the
//     activations are exactly the polled words; weight fragments are 8-byte shared loads.
//   * two extra warps per CTA do the in-leaf attention (Algorithm 2 with one key at a time):
//     each owns one (sequence, head) pair and keeps the running stats (m, l, o) of every query
//     of the leaf in shared memory.  When the pair (k_j, v_j) arrives it first finishes query
//     j+1 (the only one on the critical path) and publishes c_{j+1} = o/l, and only then folds
//     the new pair into the later queries of the leaf, while the rest of the chip is busy with
//     the mat-vecs of step j+1.  These warps also apply qkRMS to k_j and write the caches.
//   * a CTA is 384 threads = three warpgroups (MMA warps 0-3, MMA warps 4-7, the attention warps plus two idle
//     warps): once the weights are staged, setmaxnreg moves registers from the last group to the MMA warps, which
//     then hold all of a phase's fragments (up to 64 loads in flight per thread) without spilling.
#include <cuda_bf16.h>

#include <type_traits>

#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

constexpr int kMmaWarps = 8;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kAttnSlots = 2;
// Three warpgroups: MMA warps 0-3, MMA warps 4-7, and the two attention warps with two idle ones, so that registers can
// move from the last group to the MMA warps after the weights are staged (setmaxnreg works on whole warpgroups).
constexpr int kLeafMmaThreads = kMmaThreads + 128;
constexpr int kRegsMma = 216, kRegsAttn = 72;           // 2 * 128 * 216 + 128 * 72 <= 65536
constexpr int kNT = 4;                  // n-tiles (8 weight rows each) per pass
constexpr int kQStride = kHeadDim + 2;  // bf16 elements per query row in shared memory
constexpr int kOStride = kHeadDim + 1;  // floats per o row in shared memory

struct LeafMmaLayout {
  int max_nd, max_nf;          // weight rows per CTA (upper bounds): d-row matrices, W_up
  int stride_d, stride_f;      // shared-memory row strides in elements (K + 16)
  int lf;                      // leaf capacity of the attention state
  int q_smem;                  // 1: the attention warps keep a copy of the leaf's queries in shared memory; 0: they read
                               // them from global memory (what lets a 64-position leaf fit when an SM owns two pairs)
  size_t off_wo, off_wup, off_wdn, off_wk, off_wv, off_red, off_ssq, off_hown, off_attn, attn_bytes, total;
};

LeafMmaLayout leaf_mma_layout(int d, int dff, int grid, int lf, int slots, int q_smem) {
  LeafMmaLayout L;
  L.max_nd = 2 * ceil_div(d / 2, grid);
  L.max_nf = 2 * ceil_div(dff / 2, grid);
  L.stride_d = d + 16;
  L.stride_f = dff + 16;
  L.lf = lf;
  L.q_smem = q_smem;
  size_t o = 64;                                             // abort flag
  L.off_red = o;   o += sizeof(float4) * kMmaWarps * kNT * 32;
  L.off_ssq = o;   o += sizeof(float) * kMmaWarps * 16;
  L.off_hown = o;  o += align_up(sizeof(float) * 16 * (size_t)L.max_nd, 16);
  L.attn_bytes = align_up((q_smem ? (size_t)lf * kQStride * 2 : 0) + (size_t)lf * kOStride * 4 + (size_t)lf * 8 + 2 * kHeadDim * 4, 16);
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
__device__ __forceinline__ void mma_bf16(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// One weight row, global -> shared memory, as an asynchronous bulk copy that reports its bytes to an mbarrier (both
// addresses 16-byte aligned, the size a multiple of 16 bytes).
__device__ __forceinline__ void bulk_row(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void mma_warps_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory"); }

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

// What one mat-vec phase works on.  Tiles are groups of 8 weight rows in shared memory.
// Exchange words of a [B, K] bf16 vector are stored in the order the MMA fragments are read:
// [k-step of 16][16 sequence slots][4 groups of 4 k][2 words of 2 k], so that one warp-wide
// 16-byte load (8 sequences x 4 groups) covers 512 contiguous bytes.  Index of the word that
// holds elements k, k+1 (k even) of sequence b:
__device__ __forceinline__ size_t ll_word(int b, int k) {
  return ((size_t)((k >> 4) * 16 + b) * 4 + ((k & 15) >> 2)) * 2 + ((k & 3) >> 1);
}

// Sum of squares (of the raw values) and optional gain for one k-step of fragments; gp points
// at this thread's 4 gains of the k-step (or is null).
template <int MB>
__device__ __forceinline__ void frag_ssq_gain(unsigned (&a)[4], const __nv_bfloat16* gp, float& sq0, float& sq1) {
  float gn[4] = {1.f, 1.f, 1.f, 1.f};
  if (gp) {
    const uint2 gw = *reinterpret_cast<const uint2*>(gp);
    gn[0] = bf_lo(gw.x); gn[1] = bf_hi(gw.x); gn[2] = bf_lo(gw.y); gn[3] = bf_hi(gw.y);
  }
#pragma unroll
  for (int r = 0; r < MB; ++r) {
    const float v0 = bf_lo(a[r]), v1 = bf_hi(a[r]), v2 = bf_lo(a[2 + r]), v3 = bf_hi(a[2 + r]);
    const float s = v0 * v0 + v1 * v1 + v2 * v2 + v3 * v3;
    if (r == 0) sq0 += s; else sq1 += s;
    if (gp) { a[r] = pack_bf2(v0 * gn[0], v1 * gn[1]); a[2 + r] = pack_bf2(v2 * gn[2], v3 * gn[3]); }
  }
}

// Barrier over all CTAs, run by the MMA warps only (the attention warps never wait on it).
__device__ __forceinline__ bool mma_grid_barrier(SyncArea* sync, volatile int* s_abort, unsigned target) {
  mma_warps_sync();
  if (threadIdx.x == 0) {
    // the release is cumulative over what the CTA barrier above ordered before it: no separate fence
    red_release_add_u32(&sync->bar_count, 1u);
    unsigned spins = 0;
    unsigned long long t_start = 0;
    while (ld_acquire_u32(&sync->bar_count) < target) {
      if ((++spins & 255u) == 0u && wait_expired(sync, t_start)) { *s_abort = 1; break; }
    }
  }
  mma_warps_sync();
  return *s_abort == 0;
}

// ---- attention warp: one (sequence, head) pair for the whole leaf ----------------------------
// QSMEM (compile-time, like the other switches: see the kernel): the leaf's queries are copied to shared memory.
template <bool TIMERS, bool QSMEM>
__device__ void attention_role(const LeafParams& p, const LeafMmaLayout& L, unsigned char* smem_slot, int pair,
                               const unsigned long long* ll_kv, unsigned long long* ll_c) {
  const int lane = threadIdx.x & 31;
  const int B = p.B, d = p.d, H = p.H;
  const int b = pair / H, h = pair % H;
  const int Bs = p.Bs ? p.Bs : B, bc = p.b0 + b;               // row stride and column of this sequence in q / state / caches
  const int n = p.t1 - p.t0;
  __nv_bfloat16* qs = reinterpret_cast<__nv_bfloat16*>(smem_slot);
  float* os = reinterpret_cast<float*>(smem_slot + (QSMEM ? (size_t)L.lf * kQStride * 2 : 0));
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

  if (p.dec_chunks > 0) {
    // Decode step (one position): build the position's state here.  Seed: its temporary pair (logit s<q, k~>, l = 1,
    // o = v~); then the partial states of the cache's chunks (Algorithm 2 per chunk, written by the decode attention
    // kernel) are folded in chunk order.  Lane = dimensions 2 lane, 2 lane + 1.
    const size_t roff = (size_t)b * d + h * kHeadDim + 2 * lane;
    const unsigned qw = *reinterpret_cast<const unsigned*>(q + roff);
    const unsigned kw = *reinterpret_cast<const unsigned*>(reinterpret_cast<const __nv_bfloat16*>(p.kt) + roff);
    const unsigned vw = *reinterpret_cast<const unsigned*>(reinterpret_cast<const __nv_bfloat16*>(p.vt) + roff);
    float m = warp_sum(bf_lo(qw) * bf_lo(kw) + bf_hi(qw) * bf_hi(kw)) * p.scale_log2, l = 1.0f;
    float o0 = bf_lo(vw), o1 = bf_hi(vw);
    const float* part = p.dec_part + (size_t)pair * p.dec_stride * 66;
#pragma unroll 4
    for (int ch = 0; ch < p.dec_chunks; ++ch) {
      const float mc = __ldcg(part + ch * 66 + 64), lc = __ldcg(part + ch * 66 + 65);
      const float2 oc = __ldcg(reinterpret_cast<const float2*>(part + ch * 66 + 2 * lane));
      const float m_new = fmaxf(m, mc);
      const float a = exp2f(m - m_new), bb = exp2f(mc - m_new);
      o0 = o0 * a + oc.x * bb; o1 = o1 * a + oc.y * bb;
      l = l * a + lc * bb;
      m = m_new;
    }
    os[2 * lane] = o0; os[2 * lane + 1] = o1;
    if (lane == 0) { ms[0] = m; ls[0] = l; }
  } else {
  // queries and carried stats of the leaf (written by earlier kernels of this call)
  for (int i = 0; i < n; ++i) {
    const size_t row = (size_t)(p.t0 - p.row_off + i) * Bs + bc;
    if (QSMEM)
      *reinterpret_cast<unsigned*>(qs + i * kQStride + 2 * lane) =
          *reinterpret_cast<const unsigned*>(q + row * d + h * kHeadDim + 2 * lane);
    os[i * kOStride + lane] = p.st_o[row * d + h * kHeadDim + lane];
    os[i * kOStride + lane + 32] = p.st_o[row * d + h * kHeadDim + lane + 32];
  }
  for (int i = lane; i < n; i += 32) {
    const size_t row = (size_t)(p.t0 - p.row_off + i) * Bs + bc;
    ms[i] = p.st_m[row * H + h];
    ls[i] = p.st_l[row * H + h];
  }
  }
  __syncwarp();
  const float gk0 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane) : 1.0f;
  const float gk1 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane + 1) : 1.0f;
  unsigned long long* c_word = ll_c + ll_word(b, h * kHeadDim + 2 * lane);
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
    unsigned q_next = 0u;                                    // this lane's two values of query j + 1 (fetched ahead of the wait)
    if (!QSMEM && j + 1 < n)
      q_next = *reinterpret_cast<const unsigned*>(q + ((size_t)(p.t0 - p.row_off + j + 1) * Bs + bc) * d + h * kHeadDim + 2 * lane);
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
    const size_t crow = ((size_t)(p.t0 + j) * Bs + bc) * d + h * kHeadDim + 2 * lane;
    *reinterpret_cast<unsigned*>(kc + crow) = kq;
    *reinterpret_cast<unsigned*>(vc + crow) = vq;
    if (j + 1 >= n) break;
    const float kf0 = bf_lo(kq), kf1 = bf_hi(kq), vf0 = bf_lo(vq), vf1 = bf_hi(vq);
    {
      // critical path: finish query j+1 and publish c_{j+1}
      const int i = j + 1;
      const unsigned qw = QSMEM ? *reinterpret_cast<const unsigned*>(qs + i * kQStride + 2 * lane) : q_next;
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
      float s = 0.f;
      if (QSMEM) {
        const __nv_bfloat16* qi = qs + i * kQStride;
#pragma unroll 8
        for (int e = 0; e < kHeadDim; e += 2) {
          const unsigned qw = *reinterpret_cast<const unsigned*>(qi + e);
          s += bf_lo(qw) * kbuf[e] + bf_hi(qw) * kbuf[e + 1];
        }
      } else {
        const uint4* qg = reinterpret_cast<const uint4*>(q + ((size_t)(p.t0 - p.row_off + i) * Bs + bc) * d + h * kHeadDim);
        uint4 qv[8];
#pragma unroll
        for (int v = 0; v < 8; ++v) qv[v] = qg[v];
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          s += bf_lo(qv[v].x) * kbuf[8 * v] + bf_hi(qv[v].x) * kbuf[8 * v + 1] + bf_lo(qv[v].y) * kbuf[8 * v + 2] + bf_hi(qv[v].y) * kbuf[8 * v + 3] +
               bf_lo(qv[v].z) * kbuf[8 * v + 4] + bf_hi(qv[v].z) * kbuf[8 * v + 5] + bf_lo(qv[v].w) * kbuf[8 * v + 6] + bf_hi(qv[v].w) * kbuf[8 * v + 7];
        }
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

// TIMERS and GAINS are compile-time: the token step is a latency chain of code that runs once per token, and every
// instruction and live register that is compiled in costs time even when its branch is not taken.
template <int MB, bool TIMERS, bool GAINS, bool QSMEM>
__global__ void __launch_bounds__(kLeafMmaThreads, 1) leaf_mma_kernel(const LeafParams p, const LeafMmaLayout L,
                                                                      unsigned long long* ll_c, unsigned long long* ll_h,
                                                                      unsigned long long* ll_g, unsigned long long* ll_z,
                                                                      unsigned long long* ll_kv) {
  extern __shared__ __align__(128) unsigned char smem[];
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem);
  float4* red = reinterpret_cast<float4*>(smem + L.off_red);
  float* ssq_red = reinterpret_cast<float*>(smem + L.off_ssq);
  float* hown = reinterpret_cast<float*>(smem + L.off_hown);
  __nv_bfloat16* s_wo = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wo);
  __nv_bfloat16* s_wup = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wup);
  __nv_bfloat16* s_wdn = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wdn);
  __nv_bfloat16* s_wk = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wk);
  __nv_bfloat16* s_wv = reinterpret_cast<__nv_bfloat16*>(smem + L.off_wv);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int B = p.B, d = p.d, H = p.H, dff = p.dff;
  if (*reinterpret_cast<volatile unsigned*>(&p.sync->abort_flag)) return;
  // rows are dealt out in pairs so that a published word (two consecutive rows) has one owner
  const int d_lo = 2 * (int)((long long)(d / 2) * cta / G), d_hi = 2 * (int)((long long)(d / 2) * (cta + 1) / G);
  const int f_lo = 2 * (int)((long long)(dff / 2) * cta / G), f_hi = 2 * (int)((long long)(dff / 2) * (cta + 1) / G);
  const int nd = d_hi - d_lo, nf = f_hi - f_lo;

  // The CTA's weight rows go to shared memory as asynchronous bulk copies, one per row, issued by the threads of warp 0
  // and counted by an mbarrier; the attention warps, which never read the weights, do not wait for them and build the
  // leaf's state meanwhile; the MMA warps wait before their first token step.
  const uint32_t w_bar = smem_u32(smem + 8);
  if (tid == 0) {
    *s_abort = 0;
    mbar_init(w_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect_tx(w_bar, (uint32_t)(((size_t)3 * nd * d + (size_t)nf * d + (size_t)nd * dff) * 2));      // W_o, W_k, W_v; W_up; W_down
  }
  __syncthreads();
  if (warp == 0) {
    auto stage = [&](__nv_bfloat16* dst, int dst_stride, const void* src_base, int row_lo, int nrows, int K) {
      const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(src_base) + (size_t)row_lo * K;
      for (int r = lane; r < nrows; r += 32)
        bulk_row(smem_u32(dst + (size_t)r * dst_stride), src + (size_t)r * K, (uint32_t)K * 2u, w_bar);
    };
    stage(s_wo, L.stride_d, p.w_o, d_lo, nd, d);
    stage(s_wup, L.stride_d, p.w_up, f_lo, nf, d);
    stage(s_wdn, L.stride_f, p.w_down, d_lo, nd, dff);
    stage(s_wk, L.stride_d, p.w_k, d_lo, nd, d);
    stage(s_wv, L.stride_d, p.w_v, d_lo, nd, d);
  }

  if (warp >= kMmaWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsAttn));
    const int slot = warp - kMmaWarps;
    const int pair = cta + slot * G;
    if (slot < kAttnSlots && pair < B * H) attention_role<TIMERS, QSMEM>(p, L, smem + L.off_attn + (size_t)slot * L.attn_bytes, pair, ll_kv, ll_c);
    return;
  }

  // ------------------------------ MMA warps ------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsMma));
  // The four mat-vec phases of a token step run through ONE inlined copy of the code below (a loop
  // over the phase index): the step executes once per token, so four straight-line copies would
  // only thrash the instruction cache, and calls through a real function would put the fragments
  // and accumulators on the stack, where every access is an L2 round trip.
  constexpr int KC = 8;                                          // k-steps per round of loads
  const int g = lane >> 2, c = lane & 3;
  const bool pre = (p.norm_flags & RT_NORM_PRE) != 0;
  const bool kv_norm = pre && !(p.norm_flags & RT_NORM_SKIP_Z);
  const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(p.x);
  __nv_bfloat16* z = reinterpret_cast<__nv_bfloat16*>(p.z);
  // g as packed bf16 in the order the fragments are read: [k-step of 16][16 sequence slots][16 k], so the
  // 8 sequences x 32 bytes one warp-wide load touches are 256 contiguous bytes (2 lines instead of 8)
  __nv_bfloat16* g_pk = reinterpret_cast<__nv_bfloat16*>(ll_g);
  auto g_index = [](int b, int k) -> size_t { return ((size_t)((k >> 4) * 16 + b) << 4) + (size_t)(k & 15); };
  const float inv_d = 1.0f / (float)d;
  const int nt_d = (nd + 7) / 8, nt_f = (nf + 7) / 8;
  const bool has0 = g < B, has1 = (MB == 2) && (g + 8 < B);
  unsigned bar_target = p.bar_base;
  const bool timing = TIMERS && (cta == 0 && tid == 0);
  unsigned long long t_ph = timing ? globaltimer_ns() : 0ull;

  // the weight rows must have landed (the attention warps have been at work since the copies were issued); warp 0 waits
  // for the copies, the other MMA warps for warp 0
  if (warp == 0 && !mbar_wait(w_bar, 0, s_abort, p.sync)) *s_abort = 1;
  mma_warps_sync();
  if (*s_abort) return;

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
      if (ph == 2) {
        // every CTA's slice of g (packed bf16) must be complete before anyone multiplies by W_down
        bar_target += (unsigned)G;
        const unsigned long long tb = timing ? globaltimer_ns() : 0ull;
        if (!mma_grid_barrier(p.sync, s_abort, bar_target)) return;
        if (timing) wait_ns += globaltimer_ns() - tb;
      }
      const int n_ks = K / 16;
      const int ks_per_warp = (n_ks + kMmaWarps - 1) / kMmaWarps;
      const int ks0 = warp * ks_per_warp;
      const int ks1 = ks0 + ks_per_warp < n_ks ? ks0 + ks_per_warp : n_ks;

      const int tile_step = (ph == 2) ? 1 : kNT;                   // W_down: one tile per pass (see below)
      for (int t0n = 0; t0n < nt_all; t0n += tile_step) {
        const int n_tiles = nt_all - t0n < tile_step ? nt_all - t0n : tile_step;
        // rows this thread finishes after the reduction (warp w finishes tile t0n + w)
        const int ti_e = t0n + warp;
        const bool second_e = (ph == 3) && ti_e >= nt_d;
        const int rl = (second_e ? ti_e - nt_d : ti_e) * 8 + 2 * c;
        const bool mine = warp < n_tiles && rl < nrows;
        unsigned xw0 = 0, xw1 = 0;
        if (ph == 0 && mine) {                                     // x_t for the residual, fetched before the wait
          if (has0) xw0 = *reinterpret_cast<const unsigned*>(x + (size_t)g * p.x_bs + (size_t)(t - p.row_off) * p.x_ts + d_lo + rl);
          if (has1) xw1 = *reinterpret_cast<const unsigned*>(x + (size_t)(g + 8) * p.x_bs + (size_t)(t - p.row_off) * p.x_ts + d_lo + rl);
        }

        // The loops below are written without branches around the loads and the products (indices
        // are clamped, missing sequences and k-steps contribute zeros): a branch per product costs
        // more here than the product.
        float sq0 = 0.f, sq1 = 0.f;
        bool alive = true;
        const int g0 = has0 ? g : 0, g1 = has1 ? g + 8 : 0;        // rows read by lanes without a sequence (masked below)
        const unsigned keep0 = has0 ? 0xffffffffu : 0u, keep1 = has1 ? 0xffffffffu : 0u;
        if (ph == 2) {
          // W_down reads g as packed bf16 after the barrier: plain loads, and ALL of this warp's
          // k-steps are in flight before the first product (at d_ff = 4096: 32 k-steps, 64 loads when B > 8).  One tile per
          // pass keeps this at 32 products; the two accumulators halve the dependent chain.
          constexpr int KD = 32;
          float acc[2][4];
#pragma unroll
          for (int j = 0; j < 4; ++j) { acc[0][j] = acc[1][j] = 0.f; }
          // this thread's 8 bytes of weight row g (clamped to the rows that exist) of the tile, at k = 4c
          const int valid = nrows - t0n * 8 < 8 ? nrows - t0n * 8 : 8;
          const unsigned char* wd0 = reinterpret_cast<const unsigned char*>(s_wdn + (size_t)(t0n * 8 + (g < valid ? g : valid - 1)) * stride + 4 * c);
          const __nv_bfloat16* b0p = g_pk + g_index(g0, 4 * c);          // + 256 elements per k-step
          const __nv_bfloat16* b1p = g_pk + g_index(g1, 4 * c);
          for (int kc0 = ks0; kc0 < ks1; kc0 += KD) {
            unsigned ad[KD][4];
            const int n_here = ks1 - kc0;
            uint2 w0[KD], w1[MB == 2 ? KD : 1];
#pragma unroll
            for (int i = 0; i < KD; ++i) w0[i] = ld_cg_v2_if(b0p + (size_t)(kc0 + (i < n_here ? i : 0)) * 256, (i < n_here ? 1u : 0u) & keep0);
            if (MB == 2) {
#pragma unroll
              for (int i = 0; i < KD; ++i) w1[i] = ld_cg_v2_if(b1p + (size_t)(kc0 + (i < n_here ? i : 0)) * 256, (i < n_here ? 1u : 0u) & keep1);
            }
#pragma unroll
            for (int i = 0; i < KD; ++i) {
              ad[i][0] = w0[i].x; ad[i][2] = w0[i].y;
              if (MB == 2) { ad[i][1] = w1[i].x; ad[i][3] = w1[i].y; } else { ad[i][1] = 0u; ad[i][3] = 0u; }
            }
            const unsigned char* wd = wd0 + (size_t)kc0 * 32;
#pragma unroll
            for (int i = 0; i < KD; ++i) {
              const uint2 bw = *reinterpret_cast<const uint2*>(wd + (i < n_here ? i : 0) * 32);
              mma_bf16(acc[i & 1], ad[i], bw.x, bw.y);
            }
          }
          red[(warp * kNT) * 32 + lane] = make_float4(acc[0][0] + acc[1][0], acc[0][1] + acc[1][1], acc[0][2] + acc[1][2], acc[0][3] + acc[1][3]);
        } else {
        if (ks0 >= ks1) {                                          // a warp without k-steps (narrow layers) contributes zeros
          for (int nt = 0; nt < n_tiles; ++nt) red[(warp * kNT + nt) * 32 + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int kc0 = ks0; kc0 < ks1; kc0 += KC) {
          unsigned a[KC][4];
#pragma unroll
          for (int i = 0; i < KC; ++i) { a[i][0] = a[i][1] = a[i][2] = a[i][3] = 0u; }
          const int n_here = ks1 - kc0;                             // k-steps of this round (the rest stay zero)
          {
            // flag-carrying words: a k-step is 8 words per sequence, this thread takes the 2 adjacent ones at 4c
            const unsigned long long* base0 = act_ll + ll_word(g0, 4 * c) + (size_t)kc0 * 128;   // + 128 words per k-step
            const unsigned long long* base1 = act_ll + ll_word(g1, 4 * c) + (size_t)kc0 * 128;
            unsigned need0 = 0, need1 = 0;
#pragma unroll
            for (int i = 0; i < KC; ++i) {
              if (i < n_here) { need0 |= (1u << i) & keep0; need1 |= (1u << i) & keep1; }
            }
            unsigned spins = 0;
            unsigned long long t_start = 0;
            const unsigned long long t_poll = timing ? globaltimer_ns() : 0ull;
            while (alive) {
              // every outstanding word of the round is loaded (under a predicate, not a branch) before
              // any flag is looked at, so the loads overlap
              uint4 w0[KC], w1[MB == 2 ? KC : 1];
#pragma unroll
              for (int i = 0; i < KC; ++i) w0[i] = ld_relaxed_v4_if(base0 + (size_t)(i < n_here ? i : 0) * 128, (need0 >> i) & 1u);
              if (MB == 2) {
#pragma unroll
                for (int i = 0; i < KC; ++i) w1[i] = ld_relaxed_v4_if(base1 + (size_t)(i < n_here ? i : 0) * 128, (need1 >> i) & 1u);
              }
#pragma unroll
              for (int i = 0; i < KC; ++i) {
                const bool okw = (w0[i].y == seq) & (w0[i].w == seq) & ((need0 >> i) & 1u);
                a[i][0] = okw ? w0[i].x : a[i][0];
                a[i][2] = okw ? w0[i].z : a[i][2];
                need0 &= okw ? ~(1u << i) : 0xffffffffu;
              }
              if (MB == 2) {
#pragma unroll
                for (int i = 0; i < KC; ++i) {
                  const bool okw = (w1[i].y == seq) & (w1[i].w == seq) & ((need1 >> i) & 1u);
                  a[i][1] = okw ? w1[i].x : a[i][1];
                  a[i][3] = okw ? w1[i].z : a[i][3];
                  need1 &= okw ? ~(1u << i) : 0xffffffffu;
                }
              }
              if (__all_sync(0xffffffffu, (need0 | need1) == 0u)) break;
              if ((++spins & 63u) == 0u) {
                int bad = 0;
                if (lane == 0) bad = wait_expired(p.sync, t_start) ? 1 : 0;
                if (__shfl_sync(0xffffffffu, bad, 0)) { *s_abort = 1; alive = false; }
              }
            }
            if (timing) wait_ns += globaltimer_ns() - t_poll;
          }
          const __nv_bfloat16* gc = (GAINS && gp) ? gp + (size_t)kc0 * 16 : nullptr;
          if (want_ssq) {
#pragma unroll
            for (int i = 0; i < KC; ++i) frag_ssq_gain<MB>(a[i], (GAINS && gc) ? gc + (i < n_here ? i : 0) * 16 : nullptr, sq0, sq1);
          }
          // products, one tile of 8 weight rows after the other (a rolled loop: the step runs once per token, so
          // compact code counts for more than interleaving the tiles' products; two accumulators per tile halve the
          // dependent chain), each tile's partial sums going straight to the reduction buffer
#pragma unroll 1
          for (int nt = 0; nt < n_tiles; ++nt) {
            float ce[4] = {0.f, 0.f, 0.f, 0.f}, co[4] = {0.f, 0.f, 0.f, 0.f};
            const int ti = t0n + nt;
            const bool second = (ph == 3) && ti >= nt_d;
            const int r0 = (second ? ti - nt_d : ti) * 8;
            const int valid = nrows - r0 < 8 ? nrows - r0 : 8;
            const int r = r0 + (g < valid ? g : valid - 1);
            const __nv_bfloat16* wbase = (ph == 0) ? s_wo : (ph == 1) ? s_wup : (second ? s_wv : s_wk);
            const unsigned char* w = reinterpret_cast<const unsigned char*>(wbase + (size_t)r * stride + 4 * c) + (size_t)kc0 * 32;
#pragma unroll
            for (int i = 0; i < KC; ++i) {
              const uint2 bw = *reinterpret_cast<const uint2*>(w + (i < n_here ? i : 0) * 32);
              if (i & 1) mma_bf16(co, a[i], bw.x, bw.y); else mma_bf16(ce, a[i], bw.x, bw.y);
            }
            float4 v = make_float4(ce[0] + co[0], ce[1] + co[1], ce[2] + co[2], ce[3] + co[3]);
            if (kc0 > ks0) { const float4 o = red[(warp * kNT + nt) * 32 + lane]; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
            red[(warp * kNT + nt) * 32 + lane] = v;
          }
        }
        }
        // ---- reduce the K split over the 8 warps; warp w then holds the sums of tile t0n + w ----
        if (want_ssq) {
          sq0 += __shfl_xor_sync(0xffffffffu, sq0, 1); sq0 += __shfl_xor_sync(0xffffffffu, sq0, 2);
          sq1 += __shfl_xor_sync(0xffffffffu, sq1, 1); sq1 += __shfl_xor_sync(0xffffffffu, sq1, 2);
          if (c == 0) { ssq_red[warp * 16 + g] = sq0; ssq_red[warp * 16 + 8 + g] = sq1; }
        }
        mma_warps_sync();
        if (*s_abort) return;
        float y0 = 0.f, y1 = 0.f, y2 = 0.f, y3 = 0.f, ssq_lo = 0.f, ssq_hi = 0.f;
        if (warp < n_tiles) {
#pragma unroll
          for (int w = 0; w < kMmaWarps; ++w) {
            const float4 v = red[(w * kNT + warp) * 32 + lane];
            y0 += v.x; y1 += v.y; y2 += v.z; y3 += v.w;
          }
          if (want_ssq) {
#pragma unroll
            for (int w = 0; w < kMmaWarps; ++w) { ssq_lo += ssq_red[w * 16 + g]; ssq_hi += ssq_red[w * 16 + 8 + g]; }
          }
        }
        mma_warps_sync();       // red / ssq_red may be overwritten from here on
        // ---- epilogue: y0, y1 = rows rl, rl+1 for sequence g; y2, y3 = the same rows for sequence g+8 ----
        if (mine) {
          if (ph == 0) {                                            // h = x_t + alpha W_o c_t
            if (has0) {
              const float h0 = bf_lo(xw0) + p.alpha * y0, h1 = bf_hi(xw0) + p.alpha * y1;
              hown[g * L.max_nd + rl] = h0; hown[g * L.max_nd + rl + 1] = h1;
              st_relaxed_u64(ll_h + ll_word(g, d_lo + rl), pack_bf2(h0, h1), seq);
            }
            if (has1) {
              const float h0 = bf_lo(xw1) + p.alpha * y2, h1 = bf_hi(xw1) + p.alpha * y3;
              hown[(g + 8) * L.max_nd + rl] = h0; hown[(g + 8) * L.max_nd + rl + 1] = h1;
              st_relaxed_u64(ll_h + ll_word(g + 8, d_lo + rl), pack_bf2(h0, h1), seq);
            }
          } else if (ph == 1) {                                     // g = GELU(W_up RMS(h)), packed bf16
            if (has0) {
              const float rs = pre ? rsqrtf(ssq_lo * inv_d + p.eps) : 1.0f;
              *reinterpret_cast<unsigned*>(g_pk + g_index(g, f_lo + rl)) = pack_bf2(gelu_erf_f(y0 * rs), gelu_erf_f(y1 * rs));
            }
            if (has1) {
              const float rs = pre ? rsqrtf(ssq_hi * inv_d + p.eps) : 1.0f;
              *reinterpret_cast<unsigned*>(g_pk + g_index(g + 8, f_lo + rl)) = pack_bf2(gelu_erf_f(y2 * rs), gelu_erf_f(y3 * rs));
            }
          } else if (ph == 2) {                                     // z_t = h + alpha W_down g   (layer output)
            if (has0) {
              const unsigned zw = pack_bf2(hown[g * L.max_nd + rl] + p.alpha * y0, hown[g * L.max_nd + rl + 1] + p.alpha * y1);
              *reinterpret_cast<unsigned*>(z + (size_t)g * p.z_bs + (size_t)(t - p.row_off) * p.z_ts + d_lo + rl) = zw;
              st_relaxed_u64(ll_z + ll_word(g, d_lo + rl), zw, seq);
            }
            if (has1) {
              const unsigned zw = pack_bf2(hown[(g + 8) * L.max_nd + rl] + p.alpha * y2, hown[(g + 8) * L.max_nd + rl + 1] + p.alpha * y3);
              *reinterpret_cast<unsigned*>(z + (size_t)(g + 8) * p.z_bs + (size_t)(t - p.row_off) * p.z_ts + d_lo + rl) = zw;
              st_relaxed_u64(ll_z + ll_word(g + 8, d_lo + rl), zw, seq);
            }
          } else {                                                  // raw k_t, v_t from RMS(z_t): Eqs. (1)-(2) before qkRMS
            const size_t col = (size_t)(second_e ? d : 0) + d_lo + rl;
            if (has0) {
              const float rs = kv_norm ? rsqrtf(ssq_lo * inv_d + p.eps) : 1.0f;
              st_relaxed_v4(ll_kv + (size_t)g * (2 * d) + col, __float_as_uint(y0 * rs), seq, __float_as_uint(y1 * rs), seq);
            }
            if (has1) {
              const float rs = kv_norm ? rsqrtf(ssq_hi * inv_d + p.eps) : 1.0f;
              st_relaxed_v4(ll_kv + (size_t)(g + 8) * (2 * d) + col, __float_as_uint(y2 * rs), seq, __float_as_uint(y3 * rs), seq);
            }
          }
        }
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

// Picks the leaf capacity and the launch shape for a device with `sms` multiprocessors and `max_smem` bytes of shared
// memory per CTA (pure host arithmetic); returns false when this kernel does not take the shape (the generic leaf
// kernel does).
bool leaf_mma_shape(int B, int d, int H, int dff, int want_leaf, int sms, size_t max_smem, LeafMmaLaunch* out) {
  if (B > 16 || (d % 64) || (dff % 16) || B * H > kAttnSlots * sms) return false;
  const int cands[3] = {64, 32, 16};
  for (int lf : cands) {
    if (want_leaf && lf != want_leaf) continue;
    for (int q_smem = 1; q_smem >= 0; --q_smem) {              // a longer leaf without the query copy beats a shorter one with it
      const LeafMmaLayout L = leaf_mma_layout(d, dff, sms, lf, ceil_div(B * H, sms), q_smem);
      if (L.total <= max_smem) {
        out->grid = sms; out->block = kLeafMmaThreads; out->smem = L.total; out->leaf = lf; out->q_smem = q_smem;
        return true;
      }
    }
  }
  return false;
}

// The same for the current device.
bool leaf_mma_plan(int B, int d, int H, int dff, int want_leaf, LeafMmaLaunch* out) {
  int dev = 0, sms = 0, max_smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
  return leaf_mma_shape(B, d, H, dff, want_leaf, sms, (size_t)max_smem, out);
}

cudaError_t leaf_mma_launch(const LeafParams& p, const LeafMmaLaunch& l, const LeafMmaBuffers& buf, cudaStream_t s) {
  LeafMmaLayout L = leaf_mma_layout(p.d, p.dff, l.grid, l.leaf, ceil_div(p.B * p.H, l.grid), l.q_smem);
  // compile-time variants: row blocks (B > 8), per-phase timers, RMS gains present
  const bool gains = p.g_mlp != nullptr || p.g_kv != nullptr;
  auto pick2 = [&](auto mb, auto qs) -> const void* {
    constexpr int MB = decltype(mb)::value;
    constexpr bool QS = decltype(qs)::value;
    if (p.timers) return gains ? reinterpret_cast<const void*>(&leaf_mma_kernel<MB, true, true, QS>)
                               : reinterpret_cast<const void*>(&leaf_mma_kernel<MB, true, false, QS>);
    return gains ? reinterpret_cast<const void*>(&leaf_mma_kernel<MB, false, true, QS>)
                 : reinterpret_cast<const void*>(&leaf_mma_kernel<MB, false, false, QS>);
  };
  auto pick = [&](auto mb) -> const void* {
    return l.q_smem ? pick2(mb, std::true_type{}) : pick2(mb, std::false_type{});
  };
  const void* fn = p.B > 8 ? pick(std::integral_constant<int, 2>{}) : pick(std::integral_constant<int, 1>{});
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.smem);
  if (e != cudaSuccess) return e;
  LeafParams pp = p;
  LeafMmaBuffers b = buf;
  void* args[] = {(void*)&pp, (void*)&L, (void*)&b.ll_c, (void*)&b.ll_h, (void*)&b.ll_g, (void*)&b.ll_z, (void*)&b.ll_kv};
  return cudaLaunchCooperativeKernel(fn, dim3(l.grid), dim3(l.block), args, l.smem, s);
}

}  // namespace rt
