// Pre-pass projection on the 5th-generation tensor cores (bf16 storage):
//   [q | k~ | v~][m, :] = n[m, :] . [W_q | W_k | W_v]^T   with qkRMS per head on q and k~
// (first display of Sec. 2.2; Algorithm 1 line 1 and the temporary pair of line 7, for all
// positions at once).  A dense contraction: M = B*N rows, K = d, N = 3d columns.
//
// One CTA = a 128 x 128 output tile (two heads of one of the three matrices).  Warp 4 lane 0
// streams 64-wide K blocks of n and W through a 3-stage TMA ring (128-byte swizzle), warp 5
// lane 0 issues tcgen05.mma (M=128, N=128, K=16, both operands K-major) into a 128-column TMEM
// accumulator, warps 0-3 own one output row per thread: tcgen05.ld, sum of squares per head,
// gain, bf16, 16-byte stores.  Two CTAs per SM, so one tile's epilogue overlaps the other's
// main loop.  All waits are bounded (see rt_tc.cuh).
#include <cstring>

#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

constexpr int kGemmBK = 64;
constexpr int kGemmThreads = 192;
constexpr uint32_t kGemmABytes = kBM * kGemmBK * 2;        // 16 KB

// BN: output columns per CTA.  128 with a 3-stage ring (two CTAs per SM) for the sweep over all positions; 64 (one head)
// with a 6-stage ring for launches over few rows (one position of a wide batch), which then fill twice as many SMs.
template <int BN>
struct GemmSmemT {
  static constexpr int stages = BN == 64 ? 6 : 3;
  static constexpr uint32_t b_bytes = BN * kGemmBK * 2;
  static constexpr uint32_t a = 0;
  static constexpr uint32_t b = a + stages * kGemmABytes;
  static constexpr uint32_t bars = b + stages * b_bytes;               // full[], empty[], acc_ready
  static constexpr uint32_t tmem_ptr = bars + 128;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 2)
qkv_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_n, const __grid_constant__ CUtensorMap map_wq,
                   const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv,
                   const PrepassParams p, SyncArea* sync) {
  grid_dep_sync();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  using GemmSmem = GemmSmemT<BN>;
  constexpr int kGemmBN = BN, kGemmStages = GemmSmem::stages;
  constexpr uint32_t kGemmBBytes = GemmSmem::b_bytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = p.N * p.B, d = p.d;
  const int tiles_per_mat = d / kGemmBN;
  const int which = blockIdx.y / tiles_per_mat;             // 0: q, 1: k~, 2: v~
  const int col0 = (blockIdx.y % tiles_per_mat) * kGemmBN;  // first output column within the matrix
  const int m0 = blockIdx.x * kBM;
  const int n_kb = d / kGemmBK;
  if (p.mats && !((p.mats >> which) & 1)) return;          // projection not asked for (uniform per CTA)
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + GemmSmem::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + GemmSmem::tmem_ptr);
  auto full = [&](int s) { return sbase + GemmSmem::bars + 8u * (uint32_t)s; };
  auto empty = [&](int s) { return sbase + GemmSmem::bars + 8u * (uint32_t)(kGemmStages + s); };
  const uint32_t acc_ready = sbase + GemmSmem::bars + 8u * (2 * kGemmStages);

  if (tid == 0) {
    *s_abort = 0;
    for (int s = 0; s < kGemmStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(acc_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + GemmSmem::tmem_ptr), "n"(kGemmBN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const CUtensorMap* mw = which == 0 ? &map_wq : (which == 1 ? &map_wk : &map_wv);
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kGemmStages;
        if (kb >= kGemmStages) ok = mbar_wait(empty(s), ((kb / kGemmStages) - 1) & 1, s_abort, sync);
        if (!ok) break;
        mbar_expect_tx(full(s), kGemmABytes + kGemmBBytes);
        tma_load_2d(sbase + GemmSmem::a + s * kGemmABytes, &map_n, full(s), kb * kGemmBK, m0);
        tma_load_2d(sbase + GemmSmem::b + s * kGemmBBytes, mw, full(s), kb * kGemmBK, col0);
        ++issued;
      }
      if (!ok) {
        // gave up: let the copies already started land before the shared memory goes away (bounded)
        for (int i = issued > kGemmStages ? issued - kGemmStages : 0; i < issued; ++i) {
          unsigned spins = 0;
          while (!mbar_try_wait(full(i % kGemmStages), (i / kGemmStages) & 1) && ++spins < (1u << 20)) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kGemmBN, false);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kGemmStages;
        ok = mbar_wait(full(s), (kb / kGemmStages) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a0 = make_desc(sbase + GemmSmem::a + s * kGemmABytes, 16, 1024);
        const uint64_t b0 = make_desc(sbase + GemmSmem::b + s * kGemmBBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kGemmBK / 16; ++ks)
          tc_mma(tmem, a0 + 2u * ks, b0 + 2u * ks, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
        tc_commit(empty(s));                       // the stage may be refilled once these products have read it
      }
      if (ok) tc_commit(acc_ready);
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: one output row per thread ----------------
    const int row = warp * 32 + lane;
    const int m = m0 + row;
    const bool qkn = (p.norm_flags & RT_NORM_QK) != 0 && which < 2;
    const __nv_bfloat16* gain = reinterpret_cast<const __nv_bfloat16*>(which == 0 ? p.g_q : p.g_k);
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(which == 0 ? p.q : (which == 1 ? p.kt : p.vt));
    if (mbar_wait(acc_ready, 0, s_abort, sync)) {
      tc_fence_after();
      const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
      for (int hh = 0; hh < kGemmBN / kHeadDim; ++hh) {        // one head (64 columns) at a time
        uint32_t v0[32], v1[32];
        tc_ld32(t_row + (uint32_t)(hh * kHeadDim), v0);
        tc_ld32(t_row + (uint32_t)(hh * kHeadDim + 32), v1);
        tc_wait_ld();
        float rs = 1.0f;
        if (qkn) {
          float ss = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float a = __uint_as_float(v0[i]), b = __uint_as_float(v1[i]);
            ss += a * a + b * b;
          }
          rs = rsqrtf(ss * (1.0f / kHeadDim) + p.eps);
        }
        if (m < M) {
          const int c_head = col0 + hh * kHeadDim;
          uint4* dst = reinterpret_cast<uint4*>(out + (size_t)m * d + c_head);
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {                     // 8 columns = 16 bytes per store
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int e = c8 * 8 + 2 * j;
              float x0 = __uint_as_float(e < 32 ? v0[e & 31] : v1[e & 31]) * rs;
              float x1 = __uint_as_float(e + 1 < 32 ? v0[(e + 1) & 31] : v1[(e + 1) & 31]) * rs;
              if (qkn && gain) { x0 *= __bfloat162float(gain[c_head + e]); x1 *= __bfloat162float(gain[c_head + e + 1]); }
              const __nv_bfloat162 pk = __floats2bfloat162_rn(x0, x1);
              w[j] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            dst[c8] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kGemmBN) : "memory");
  }
}

static_assert(kGemmBK == 64, "tensor_map_rows_bf16 encodes 64-column boxes");

bool qkv_gemm_tc_supported(const PrepassParams& p) { return p.d % 128 == 0 && p.d >= 128; }

cudaError_t qkv_gemm_tc_launch(const PrepassParams& p, SyncArea* sync, cudaStream_t s) {
  const int M = p.N * p.B;
  if (!p.mats && dense_qkv_pair_supported(M, p.d)) {
    // all three projections over many rows: persistent CTA pairs
    DenseParams dp;
    memset(&dp, 0, sizeof(dp));
    dp.M = M; dp.N = p.d; dp.K = p.d; dp.B = p.B; dp.epi = DENSE_QKV; dp.chained = p.chained;
    dp.A = p.n; dp.W = p.w_q; dp.W2 = p.w_k; dp.W3 = p.w_v;
    dp.q_out = p.q; dp.k_out = p.kt; dp.v_out = p.vt; dp.g_q = p.g_q; dp.g_k = p.g_k;
    dp.qk_norm = (p.norm_flags & RT_NORM_QK) ? 1 : 0; dp.qk_eps = p.eps;
    return dense_qkv_pair_launch(dp, sync, s);
  }
  int mats = 0;
  for (int w = 0; w < 3; ++w) mats += (!p.mats || ((p.mats >> w) & 1)) ? 1 : 0;
  // few rows: one head per CTA, so that the launch fills the multiprocessors
  const int bn = ceil_div(M, kBM) * mats * (p.d / 128) < sm_count() / 2 ? 64 : 128;
  CUtensorMap mn, mq, mk, mv;
  if (!tensor_map_rows_bf16(&mn, p.n, M, p.d, kBM) || !tensor_map_rows_bf16(&mq, p.w_q, p.d, p.d, bn) ||
      !tensor_map_rows_bf16(&mk, p.w_k, p.d, p.d, bn) || !tensor_map_rows_bf16(&mv, p.w_v, p.d, p.d, bn))
    return cudaErrorInvalidValue;
  dim3 grid(ceil_div(M, kBM), 3 * (p.d / bn));
  auto run = [&](auto kern, size_t smem) -> cudaError_t {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), (int)smem);
    if (e != cudaSuccess) return e;
    return launch_chained(kern, grid, dim3(kGemmThreads), smem, s, p.chained != 0, mn, mq, mk, mv, p, sync);
  };
  if (bn == 64) return run(qkv_gemm_tc_kernel<64>, GemmSmemT<64>::total + 1024);
  return run(qkv_gemm_tc_kernel<128>, GemmSmemT<128>::total + 1024);
}

}  // namespace rt
