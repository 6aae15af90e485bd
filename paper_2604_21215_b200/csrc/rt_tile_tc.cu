// Cross-block tile on the 5th-generation tensor cores (bf16 storage): Algorithm 2 (UpdateTile)
// for queries [q0,q1) against the revealed pairs [k0,k1), every sequence and head, with the
// running stats (m, l, o) carried in fp32 in the workspace.
//
// One CTA = one query tile of 128 rows of one (sequence, head) pair, looping over 64-key blocks:
//   TMA     (warp 5) the Q tile once, then K and V blocks through a 2-stage ring, straight out of
//           the position-major buffers (a 4-D tensor map picks the head's 64 columns of each row),
//           128-byte swizzle = the tensor cores' canonical shared-memory layout
//   S       (warp 4) tcgen05.mma  S[128x64] = Q . K^T  into the S columns of TMEM
//   softmax (warps 0-3, one thread per query row) tcgen05.ld of the row, block max,
//           p = 2^(s - m), row sum; P goes back into TMEM as packed bf16 over the first half of
//           the S columns it came from (tcgen05.st).  The special-function unit (16 exponentials
//           per clock and SM) is the busiest unit of this loop at d_h = 64, so a quarter of the
//           exponentials are computed on the FMA pipe instead (exp_half below)
//   PV      (warp 4) tcgen05.mma  O[128x64] += P . V  (A from TMEM, B = V MN-major: V rows are
//           keys), ACCUMULATING in the O columns of TMEM
// The running output never visits registers inside the loop: O is seeded from the carried state
// before the first block and read back once after the last.  The reference maximum m is raised
// only when a block's maximum exceeds it by more than 2^8 (the merge of Algorithm 2 is exact for
// any reference value; the bound keeps p <= 256), and then the row's O and l are rescaled in place.
// The state is renormalised to the true running maximum when it is written back, so the stored
// triple is the one Algorithm 2 defines.
// TMEM: S [0,64) O [64,128); 48 KB of shared memory and 256 threads at 64 registers, so four CTAs share
// an SM and their chains (softmax -> P.V -> S -> softmax) interleave on the tensor pipe; the threads form two
// warpgroups (softmax; issuing warps plus two idle ones) so that registers can move between them.
// Every mbarrier wait is bounded: on expiry the CTA records RT_ERR_TIMEOUT, stops issuing work,
// waits (bounded) for its copies in flight, frees its TMEM and returns.
#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

constexpr int kBK = 64;                // keys per block
constexpr uint32_t kKVBytes = kBK * kHeadDim * 2;    // 8 KB
constexpr uint32_t kQBytes = kBM * kHeadDim * 2;     // 16 KB
constexpr float kLazyLog2 = 8.0f;      // the reference maximum may lag the true one by this much (log2 units)

// Which pairs of a row's values (by pair index mod 8) take their exponentials from the FMA pipe: a quarter.  Measured on
// the c3 shape at P = 2048 / 4096 (TF/s): none 581 / 703 (all on the special-function unit, scalar arithmetic),
// 1/4 605 / 744, 3/8 594 / 720, 1/2 579 / 693.
constexpr unsigned kEmuMask = 0x88u;
constexpr int kRegsSoftmax = 88, kRegsIssue = 40;      // registers per thread after the hand-over (setmaxnreg), see the kernel
// Packed fp32 pairs (f32x2 arithmetic of sm_100): one instruction works on both halves of a 64-bit register, which
// halves the issue slots of the scale-and-subtract and of the row sum.
__device__ __forceinline__ uint64_t pk2(uint32_t lo, uint32_t hi) { uint64_t r; asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "r"(lo), "r"(hi)); return r; }
__device__ __forceinline__ uint64_t pk2f(float lo, float hi) { return pk2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void upk2(uint64_t v, uint32_t& lo, uint32_t& hi) { asm("mov.b64 {%0,%1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) { uint64_t d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) { uint64_t d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) { uint64_t d; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ float max3(float a, float b, float c) { float d; asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d; }

// p = 2^(s * scale + neg_m) for the 16 pairs of `s`, packed bf16 into w, the pairs' sums added to sum2[0..1].
// Pairs whose bit is set in kEmuMask (by pair index mod 8) take the exponential from the FMA pipe instead of the
// special-function unit: x is split into an integer j (round to nearest through the 1.5 * 2^23 constant) and r in
// [-0.5, 0.5], 2^r is a cubic (max. relative error 7.5e-5, far below the bf16 rounding of P), and j goes into the
// exponent field by an integer add.  x is clamped at -125 so that the exponent field cannot wrap.
__device__ __forceinline__ void exp_half(const uint32_t (&s)[32], float scale, float neg_m, uint32_t (&w)[16], uint64_t (&sum2)[2]) {
  const uint64_t sc2 = pk2f(scale, scale), nm2 = pk2f(neg_m, neg_m);
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const uint64_t x2 = fma2(pk2(s[2 * j], s[2 * j + 1]), sc2, nm2);
    uint32_t x0, x1, p0, p1;
    upk2(x2, x0, x1);
    if ((kEmuMask >> (j & 7)) & 1u) {
      const uint64_t magic2 = pk2f(12582912.f, 12582912.f);
      const uint64_t xc2 = pk2f(fmaxf(__uint_as_float(x0), -125.f), fmaxf(__uint_as_float(x1), -125.f));
      const uint64_t t2 = add2(xc2, magic2);
      const uint64_t r2 = sub2(xc2, sub2(t2, magic2));
      uint64_t q2 = fma2(r2, pk2f(0.0551716685f, 0.0551716685f), pk2f(0.242611125f, 0.242611125f));
      q2 = fma2(q2, r2, pk2f(0.693260968f, 0.693260968f));
      q2 = fma2(q2, r2, pk2f(0.999928057f, 0.999928057f));
      uint32_t q0, q1, t0, t1;
      upk2(q2, q0, q1);
      upk2(t2, t0, t1);
      p0 = q0 + (t0 << 23);
      p1 = q1 + (t1 << 23);
    } else {
      p0 = __float_as_uint(ex2(__uint_as_float(x0)));
      p1 = __float_as_uint(ex2(__uint_as_float(x1)));
    }
    sum2[j & 1] = add2(sum2[j & 1], pk2(p0, p1));
    const __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(p0), __uint_as_float(p1));
    w[j] = *reinterpret_cast<const uint32_t*>(&pk);
  }
}

struct TcCfg {
  static constexpr int stages = 2;
  static constexpr int ctas_per_sm = 4;
  static constexpr int threads = 8 * 32;                 // warpgroup 0: 4 softmax warps; warpgroup 1: MMA warp, TMA warp, two idle warps
  static constexpr int tmem_cols = 128;
  // offsets from a 1024-byte aligned base
  static constexpr uint32_t q = 0;
  static constexpr uint32_t k = q + kQBytes;
  static constexpr uint32_t v = k + stages * kKVBytes;
  static constexpr uint32_t bars = v + stages * kKVBytes;
  static constexpr uint32_t tmem_ptr = bars + 8 * 24;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};
enum { BAR_KV_FULL = 0, BAR_KV_EMPTY = 2, BAR_Q_FULL = 4, BAR_S_READY = 5, BAR_P_READY = 6 };

// ALIBI / CAUSAL are compile-time so that the plain kernel carries none of their registers or instructions
// (four CTAs per SM leave its softmax threads 88 registers, and it loses up to a fifth of its rate to a few spills).
template <bool ALIBI, bool CAUSAL>
__global__ void __launch_bounds__(TcCfg::threads, TcCfg::ctas_per_sm)
tile_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const TileParams p, SyncArea* sync) {
  using C = TcCfg;
  constexpr int kStages = C::stages;
  constexpr int kMmaWarp = 4, kTmaWarp = 5;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  // copy blockIdx.z of the tile (one level of Algorithm 1 in one launch); the few values derived from it are
  // recomputed where they are used rather than kept in registers across the roles
  auto shift = [&]() { return (int)blockIdx.z * p.batch_stride; };
  auto q_end = [&]() { const int q1 = p.q1 + shift(); return (p.q_limit > 0 && q1 > p.q_limit) ? p.q_limit : q1; };
  // (whole causal prefix in one launch: the CTAs with the most key blocks come first)
  const int bx = (CAUSAL && p.causal_full) ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
  const int qb = p.q0 + shift() + bx * kBM;               // first query row of this CTA
  if (qb >= q_end()) return;                              // nothing left of this copy (uniform per CTA)
  int n_blocks = (p.k1 - p.k0) / kBK;                     // whole blocks only (checked by the launcher)
  if (CAUSAL && p.causal_full) {                          // no key block beyond this CTA's own queries
    const int own = (qb + kBM - (p.k0 + shift())) / kBK;
    n_blocks = own < n_blocks ? own : n_blocks;
  }
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + C::tmem_ptr);
  auto bar = [&](int i) { return sbase + C::bars + 8u * (uint32_t)i; };

  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < kStages; ++i) { mbar_init(bar(BAR_KV_FULL + i), 1); mbar_init(bar(BAR_KV_EMPTY + i), 1); }
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_S_READY), 1);
    mbar_init(bar(BAR_P_READY), 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + C::tmem_ptr), "n"(C::tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // Registers move from the issuing warpgroup to the softmax warpgroup: the launch gives each of the 256 threads 64
  // (four CTAs per SM), the issuing warps keep kRegsIssue and the softmax warps grow to kRegsSoftmax, where their loop
  // runs without spills.  Measured (TF/s at P = 2048 / 4096): 88 + 40 628 / 769, 96 + 32 553 / 693, 104 + 24 517 / 654
  // (the issuing threads then spill), against 601 / 740 for 192 threads at 80 registers.

  if (warp >= 6) {
    // idle warps of the issuing warpgroup
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
  } else if (warp == kTmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      const int k0 = p.k0 + shift();
      mbar_expect_tx(bar(BAR_Q_FULL), kQBytes);
      tma_load_4d(sbase + C::q, &map_q, bar(BAR_Q_FULL), 0, h, b, qb);
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < n_blocks && ok; ++kb) {
        const int st = kb % kStages;
        if (kb >= kStages) ok = mbar_wait(bar(BAR_KV_EMPTY + st), ((kb / kStages) - 1) & 1, s_abort, sync);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_KV_FULL + st), 2 * kKVBytes);
        tma_load_4d(sbase + C::k + st * kKVBytes, &map_k, bar(BAR_KV_FULL + st), 0, h, b, k0 + kb * kBK);
        tma_load_4d(sbase + C::v + st * kKVBytes, &map_v, bar(BAR_KV_FULL + st), 0, h, b, k0 + kb * kBK);
        ++issued;
      }
      if (!ok) {
        // gave up: let the copies already started land before the shared memory goes away (bounded)
        unsigned spins = 0;
        while (!mbar_try_wait(bar(BAR_Q_FULL), 0) && ++spins < (1u << 20)) {}
        for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i) {
          spins = 0;
          while (!mbar_try_wait(bar(BAR_KV_FULL + i % kStages), (i / kStages) & 1) && ++spins < (1u << 20)) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(kBK, false);
      constexpr uint32_t idesc_pv = make_idesc(kHeadDim, true);
      // S(kb) = Q . K(kb)^T over the S columns (both operands K-major: 32 bytes along K per step)
      auto issue_s = [&](int kb) {
        const int st = kb % kStages;
        const uint64_t q_desc = make_desc(sbase + C::q, 16, 1024);
        const uint64_t k_desc = make_desc(sbase + C::k + st * kKVBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)
          tc_mma(tmem, q_desc + 2u * ks, k_desc + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
      };
      bool ok = mbar_wait(bar(BAR_Q_FULL), 0, s_abort, sync);
      if (ok) ok = mbar_wait(bar(BAR_KV_FULL), 0, s_abort, sync);
      if (ok) {
        tc_fence_after();
        issue_s(0);
        tc_commit(bar(BAR_S_READY));
      }
      for (int kb = 0; kb < n_blocks && ok; ++kb) {
        const int st = kb % kStages;
        const bool more = kb + 1 < n_blocks;
        if (more) ok = mbar_wait(bar(BAR_KV_FULL + (kb + 1) % kStages), ((kb + 1) / kStages) & 1, s_abort, sync);
        if (ok) ok = mbar_wait(bar(BAR_P_READY), kb & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        const uint64_t v_desc = make_desc(sbase + C::v + st * kKVBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kBK / 16; ++ks)                 // A: P in TMEM, 8 columns per step; B (MN-major): 16 key rows = 2048 bytes
          tc_mma_ts(tmem + 64u, tmem + 8u * ks, v_desc + 128u * ks, idesc_pv, 1u);
        tc_commit(bar(BAR_KV_EMPTY + st));                    // K(kb) and V(kb) have been used
        if (more) issue_s(kb + 1);                            // P(kb) has been read by then: the pipe runs in issue order
        tc_commit(bar(BAR_S_READY));                          // S(kb+1) ready, and O holds blocks 0..kb
      }
    }
    __syncwarp();
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    // ------------------------------ softmax warps: one thread per query row ------------------------------
    const int row = warp * 32 + lane;
    const int qi = qb + row;
    const bool row_ok = qi < q_end();
    const uint32_t t_s = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_o = t_s + 64u;
    const size_t sidx = (size_t)(row_ok ? qi : p.q0) * p.B + b;
    float m_used = p.st_m[sidx * p.H + h];                   // reference maximum of l and O (log2 units)
    const float slope_l2 = ALIBI ? p.alibi[h] * kLog2e : 0.f;
    const float step_raw = slope_l2 / p.scale_log2;          // slope per column, in units of the raw product
    float m_true = m_used;                                   // running maximum
    float l_run = p.st_l[sidx * p.H + h];
    uint32_t s0[32], s1[32];
    {
      // seed O with the carried output
      const uint4* src = reinterpret_cast<const uint4*>(p.st_o + sidx * p.d + h * kHeadDim);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint4 a = src[i], c = src[8 + i];
        s0[4 * i] = a.x; s0[4 * i + 1] = a.y; s0[4 * i + 2] = a.z; s0[4 * i + 3] = a.w;
        s1[4 * i] = c.x; s1[4 * i + 1] = c.y; s1[4 * i + 2] = c.z; s1[4 * i + 3] = c.w;
      }
      tc_st32(t_o, s0);
      tc_st32(t_o + 32u, s1);
    }
    bool ok = true;
    for (int kb = 0; kb < n_blocks; ++kb) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_S_READY), kb & 1, s_abort, sync));
      if (!ok) break;
      tc_fence_after();
      // ALiBi distances: the logit of this row's query (position qi) on key j gets -slope (qi - j)
      // = base + slope * column: the column part goes into the raw products (divided by the scale that is
      // applied below), the row constant into the maximum and the exponent offset.  Causal launches turn the
      // pairs at or beyond the row's position into -inf (p = 0).
      float base_l2 = 0.f;
      if (ALIBI) base_l2 = -slope_l2 * (float)(qi - (p.k0 + shift() + kb * kBK));
      auto adjust = [&](uint32_t (&v)[32], int col0) {
        if (ALIBI) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(fmaf(step_raw, (float)(i + col0), __uint_as_float(v[i])));
        }
        if (CAUSAL && p.k0 + shift() + (kb + 1) * kBK > qb) {          // (blocks wholly before the tile's first query need no mask)
          const int n_valid = qi - (p.k0 + shift() + kb * kBK);
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i + col0 >= n_valid) v[i] = 0xff800000u;
        }
      };
      // The row lives in registers half at a time (32 of its 64 values): the second half is read for the
      // maximum, dropped, and read again for the exponentials.  A TMEM load costs little; holding all 64
      // values next to the packed P words would not fit the 88 registers four resident CTAs leave a softmax thread.
      float mx4[4];                                            // four independent chains
      tc_ld32(t_s + 32u, s1);
      tc_wait_ld();
      adjust(s1, 32);
#pragma unroll
      for (int j = 0; j < 4; ++j) mx4[j] = fmaxf(__uint_as_float(s1[2 * j]), __uint_as_float(s1[2 * j + 1]));
#pragma unroll
      for (int i = 4; i < 16; ++i) mx4[i & 3] = max3(mx4[i & 3], __uint_as_float(s1[2 * i]), __uint_as_float(s1[2 * i + 1]));
      tc_ld32(t_s, s0);
      tc_wait_ld();
      adjust(s0, 0);
#pragma unroll
      for (int i = 0; i < 16; ++i) mx4[i & 3] = max3(mx4[i & 3], __uint_as_float(s0[2 * i]), __uint_as_float(s0[2 * i + 1]));
      float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      if (ALIBI) mx += base_l2;
      m_true = fmaxf(m_true, mx);
      const bool raise = mx > m_used + kLazyLog2;
      const float m_new = raise ? m_true : m_used;
      const float corr = ex2(m_used - m_new);                  // 1 when the reference stays
      float neg_m = -m_new;
      if (ALIBI) neg_m += base_l2;
      uint64_t sum2[2] = {0ull, 0ull};
      // p = 2^(s*scale - m) as packed bf16, written over the first 32 columns of the S buffer
      uint32_t w[16];
      exp_half(s0, p.scale_log2, neg_m, w, sum2);
      tc_ld32(t_s + 32u, s1);                                  // columns 32..63 are still the raw products
      tc_st16(t_s, w);
      tc_wait_ld();
      adjust(s1, 32);
      exp_half(s1, p.scale_log2, neg_m, w, sum2);
      tc_st16(t_s + 16u, w);
      {
        uint32_t a0, a1;
        upk2(add2(sum2[0], sum2[1]), a0, a1);
        l_run = l_run * corr + (__uint_as_float(a0) + __uint_as_float(a1));
      }
      m_used = m_new;
      if (__any_sync(0xffffffffu, raise)) {
        // rare: rescale this warp's rows of O in place (O is quiescent: S_READY(kb) covers P.V(kb-1))
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          tc_ld32(t_o + 32u * half, s0);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) s0[i] = __float_as_uint(__uint_as_float(s0[i]) * corr);
          tc_st32(t_o + 32u * half, s0);
        }
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_P_READY));
    }
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_S_READY), n_blocks & 1, s_abort, sync));
    if (ok) {
      tc_fence_after();
      tc_ld32(t_o, s0);
      tc_ld32(t_o + 32u, s1);
      tc_wait_ld();
      tc_fence_before();
      if (row_ok) {
        const float c = ex2(m_used - m_true);                  // back to the true maximum
        p.st_m[sidx * p.H + h] = m_true;
        p.st_l[sidx * p.H + h] = l_run * c;
        float4* dst = reinterpret_cast<float4*>(p.st_o + sidx * p.d + h * kHeadDim);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          dst[i] = make_float4(__uint_as_float(s0[4 * i]) * c, __uint_as_float(s0[4 * i + 1]) * c,
                               __uint_as_float(s0[4 * i + 2]) * c, __uint_as_float(s0[4 * i + 3]) * c);
          dst[8 + i] = make_float4(__uint_as_float(s1[4 * i]) * c, __uint_as_float(s1[4 * i + 1]) * c,
                                   __uint_as_float(s1[4 * i + 2]) * c, __uint_as_float(s1[4 * i + 3]) * c);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(C::tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------ host

static bool make_map_uncached(CUtensorMap* map, const void* base, int rows, int B, int H, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)H, (cuuint64_t)B, (cuuint64_t)rows};
  const cuuint64_t strides[3] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)H * kHeadDim * 2, (cuuint64_t)B * H * kHeadDim * 2};
  const cuuint32_t box[4] = {(cuuint32_t)kHeadDim, 1, 1, (cuuint32_t)box_rows};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows, B, H, 64] bf16 viewed as a 4-D tensor; a box is `box_rows` rows of one head of one sequence.  An encoded
// map is a pure function of these arguments, so each thread remembers the ones it made: a prefill launches a tile
// after every leaf, always on the same three buffers.
static bool make_map(CUtensorMap* map, const void* base, int rows, int B, int H, int box_rows) {
  struct Entry { const void* base; int rows, B, H, box_rows; CUtensorMap map; };
  constexpr int kEntries = 64;
  thread_local Entry tab[kEntries];
  thread_local int used = 0, next = 0;
  for (int i = 0; i < used; ++i)
    if (tab[i].base == base && tab[i].rows == rows && tab[i].B == B && tab[i].H == H && tab[i].box_rows == box_rows) {
      *map = tab[i].map;
      return true;
    }
  if (!make_map_uncached(map, base, rows, B, H, box_rows)) return false;
  const int slot = used < kEntries ? used++ : (next++ % kEntries);
  tab[slot].base = base; tab[slot].rows = rows; tab[slot].B = B; tab[slot].H = H; tab[slot].box_rows = box_rows; tab[slot].map = *map;
  return true;
}

// rows_q / rows_kv: number of rows the query buffer / caches hold (bounds for the tensor maps).
cudaError_t tile_tc_launch(const TileParams& p, int rows_q, int rows_kv, SyncArea* sync, cudaStream_t s) {
  const int nq = p.q1 - p.q0;
  if (nq <= 0 || p.k1 <= p.k0) return cudaSuccess;
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, p.q, rows_q, p.B, p.H, kBM) || !make_map(&mk, p.k_cache, rows_kv, p.B, p.H, kBK) ||
      !make_map(&mv, p.v_cache, rows_kv, p.B, p.H, kBK))
    return cudaErrorInvalidValue;
  const size_t smem = TcCfg::total + 1024;
  dim3 grid(ceil_div(nq, kBM), p.B * p.H, p.batch > 1 ? p.batch : 1);
  auto go = [&](auto kernel) -> cudaError_t {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, TcCfg::threads, smem, s>>>(mq, mk, mv, p, sync);
    return cudaGetLastError();
  };
  const bool alibi = p.alibi != nullptr, causal = p.causal != 0;
  if (alibi && causal) return go(tile_tc_kernel<true, true>);
  if (alibi) return go(tile_tc_kernel<true, false>);
  if (causal) return go(tile_tc_kernel<false, true>);
  return go(tile_tc_kernel<false, false>);
}

}  // namespace rt
