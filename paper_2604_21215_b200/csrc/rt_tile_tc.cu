// Cross-block tile on the 5th-generation tensor cores (bf16 storage): Algorithm 2 (UpdateTile)
// for queries [q0,q1) against the revealed pairs [k0,k1), every sequence and head, with the
// running stats (m, l, o) carried in fp32 in the workspace.
//
// One CTA = 128 query rows of one (sequence, head) pair, looping over 64-key blocks:
//   Q       each softmax thread loads its query row and parks it in TMEM (32 columns of packed bf16)
//   TMA     (warp 5) K and V blocks through a 4-stage ring, straight out of the position-major
//           cache (a 4-D tensor map picks the head's 64 columns of each row), 128-byte swizzle =
//           the tensor cores' canonical shared-memory layout
//   S       (warp 4) tcgen05.mma  S[128x64] = Q . K^T   (A from TMEM, B K-major from shared memory)
//   softmax (warps 0-3, one thread per query row) tcgen05.ld of the row, running max in log2
//           units, p = 2^(s - m), row sum; P goes back into TMEM as packed bf16 over the first
//           half of the S buffer it came from (tcgen05.st)
//   PV      (warp 4) tcgen05.mma  PV[128x64] = P . V  (A from TMEM, B = V MN-major: V rows are keys)
//   merge   o = o * 2^(m_old - m_new) + PV in registers (fp32), one block late
// Both products take their 128-row operand from TMEM: with N = 64 the shared-memory fetch of a
// 128x16 A slice per instruction (4 KB for 131 k MACs) was what bounded the tensor pipe, not its
// math rate.  S is double-buffered (S(kb+1) is issued while softmax(kb) runs) and the product P.V
// of block kb is folded into o during block kb+1.  TMEM: S0 [0,64) S1 [64,128) PV [128,192)
// Q [192,224); two CTAs per SM.  Every mbarrier wait is bounded: on expiry the CTA records
// RT_ERR_TIMEOUT, stops issuing work, waits (bounded) for its copies in flight, frees its TMEM and
// returns.
#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

constexpr int kBK = 64;                // keys per block
constexpr int kKvStages = 4;
constexpr int kTcThreads = 192;        // 4 softmax warps + MMA warp + TMA warp
constexpr int kTmemCols = 256;
constexpr uint32_t kColPV = 128, kColQ = 192;
constexpr uint32_t kKVBytes = kBK * kHeadDim * 2;    // 8 KB

struct TcSmem {                        // offsets from a 1024-byte aligned base
  static constexpr uint32_t k = 0;
  static constexpr uint32_t v = k + kKvStages * kKVBytes;
  static constexpr uint32_t bars = v + kKvStages * kKVBytes;
  static constexpr uint32_t tmem_ptr = bars + 128;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};
// P_READY has one barrier per S/P buffer: a softmax warp may run one block ahead of another, and its
// arrival for block kb+1 must not count towards block kb.
enum { BAR_KV_FULL = 0, BAR_KV_EMPTY = 4, BAR_Q_READY = 8, BAR_S_READY = 9, BAR_P_READY = 11, BAR_PV_READY = 13, BAR_PV_FREE = 14 };

__global__ void __launch_bounds__(kTcThreads, 2)
tile_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const TileParams p,
               SyncArea* sync) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  const int qb = p.q0 + blockIdx.x * kBM;                 // first query row of this CTA
  const int n_blocks = (p.k1 - p.k0) / kBK;               // whole blocks only (checked by the launcher)
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + TcSmem::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + TcSmem::tmem_ptr);
  auto bar = [&](int i) { return sbase + TcSmem::bars + 8u * (uint32_t)i; };

  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < kKvStages; ++i) { mbar_init(bar(BAR_KV_FULL + i), 1); mbar_init(bar(BAR_KV_EMPTY + i), 1); }
    mbar_init(bar(BAR_Q_READY), 4);
    mbar_init(bar(BAR_S_READY), 1); mbar_init(bar(BAR_S_READY + 1), 1);
    mbar_init(bar(BAR_P_READY), 4); mbar_init(bar(BAR_P_READY + 1), 4);
    mbar_init(bar(BAR_PV_READY), 1);
    mbar_init(bar(BAR_PV_FREE), 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + TcSmem::tmem_ptr), "n"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (warp == 5) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < n_blocks && ok; ++kb) {
        const int st = kb % kKvStages;
        if (kb >= kKvStages) ok = mbar_wait(bar(BAR_KV_EMPTY + st), ((kb / kKvStages) - 1) & 1, s_abort, sync);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_KV_FULL + st), 2 * kKVBytes);
        tma_load_4d(sbase + TcSmem::k + st * kKVBytes, &map_k, bar(BAR_KV_FULL + st), 0, h, b, p.k0 + kb * kBK);
        tma_load_4d(sbase + TcSmem::v + st * kKVBytes, &map_v, bar(BAR_KV_FULL + st), 0, h, b, p.k0 + kb * kBK);
        ++issued;
      }
      if (!ok) {
        // gave up: let the copies already started land before the shared memory goes away (bounded)
        for (int i = issued > kKvStages ? issued - kKvStages : 0; i < issued; ++i) {
          unsigned spins = 0;
          while (!mbar_try_wait(bar(BAR_KV_FULL + i % kKvStages), (i / kKvStages) & 1) && ++spins < (1u << 20)) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 4) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(kBK, false);
      constexpr uint32_t idesc_pv = make_idesc(kHeadDim, true);
      auto issue_s = [&](int kb) -> bool {
        const int st = kb % kKvStages, sb = kb & 1;
        if (!mbar_wait(bar(BAR_KV_FULL + st), (kb / kKvStages) & 1, s_abort, sync)) return false;
        // the S buffer also carried P(kb-2): it is free once the product P.V of block kb-2 has run
        if (kb >= 2 && !mbar_wait(bar(BAR_PV_READY), (kb - 2) & 1, s_abort, sync)) return false;
        tc_fence_after();
        const uint64_t k_desc = make_desc(sbase + TcSmem::k + st * kKVBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)            // A: 8 TMEM columns (16 bf16) per step; B: 32 bytes along K
          tc_mma_ts(tmem + (uint32_t)(sb * kBK), tmem + kColQ + 8u * ks, k_desc + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
        tc_commit(bar(BAR_S_READY + sb));
        return true;
      };
      bool ok = mbar_wait(bar(BAR_Q_READY), 0, s_abort, sync);
      if (ok) ok = issue_s(0);
      for (int kb = 0; kb < n_blocks && ok; ++kb) {
        if (kb + 1 < n_blocks) { ok = issue_s(kb + 1); if (!ok) break; }   // runs under softmax(kb)
        const int st = kb % kKvStages, sb = kb & 1;
        ok = mbar_wait(bar(BAR_P_READY + sb), (kb >> 1) & 1, s_abort, sync);
        if (ok && kb >= 1) ok = mbar_wait(bar(BAR_PV_FREE), (kb - 1) & 1, s_abort, sync);   // PV(kb-1) has been read out
        if (!ok) break;
        tc_fence_after();
        const uint64_t v_desc = make_desc(sbase + TcSmem::v + st * kKVBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kBK / 16; ++ks)                 // A: P in TMEM, 8 columns per step; B (MN-major): 16 key rows = 2048 bytes
          tc_mma_ts(tmem + kColPV, tmem + (uint32_t)(sb * kBK) + 8u * ks, v_desc + 128u * ks, idesc_pv, ks > 0 ? 1u : 0u);
        tc_commit(bar(BAR_PV_READY));
        tc_commit(bar(BAR_KV_EMPTY + st));
      }
    }
    __syncwarp();
  } else {
    // ------------------------------ softmax warps: one thread per query row ------------------------------
    const int row = warp * 32 + lane;
    const int qi = qb + row;
    const bool row_ok = qi < p.q1;
    const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
    const size_t sidx = (size_t)(row_ok ? qi : p.q0) * p.B + b;
    {
      // this row of Q: 64 bf16 = 32 packed words, parked in TMEM for the S products
      const uint4* qsrc = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.q) + sidx * p.d + h * kHeadDim);
      uint32_t qa[16], qc[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 a = qsrc[i], c = qsrc[4 + i];
        qa[4 * i] = a.x; qa[4 * i + 1] = a.y; qa[4 * i + 2] = a.z; qa[4 * i + 3] = a.w;
        qc[4 * i] = c.x; qc[4 * i + 1] = c.y; qc[4 * i + 2] = c.z; qc[4 * i + 3] = c.w;
      }
      tc_st16(t_row + kColQ, qa);
      tc_st16(t_row + kColQ + 16u, qc);
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_Q_READY));
    }
    float m_run = p.st_m[sidx * p.H + h];
    float l_run = p.st_l[sidx * p.H + h];
    float o[kHeadDim];
    {
      const float4* src = reinterpret_cast<const float4*>(p.st_o + sidx * p.d + h * kHeadDim);
#pragma unroll
      for (int i = 0; i < kHeadDim / 4; ++i) {
        const float4 v = src[i];
        o[4 * i] = v.x; o[4 * i + 1] = v.y; o[4 * i + 2] = v.z; o[4 * i + 3] = v.w;
      }
    }
    float corr_prev = 1.0f;
    bool ok = true;
    for (int kb = 0; kb < n_blocks; ++kb) {
      const int sb = kb & 1;
      ok = mbar_wait(bar(BAR_S_READY + sb), (kb >> 1) & 1, s_abort, sync);
      if (!ok) break;
      tc_fence_after();
      uint32_t s0[32], s1[32];
      tc_ld32(t_row + (uint32_t)(sb * kBK), s0);
      tc_ld32(t_row + (uint32_t)(sb * kBK + 32), s1);
      tc_wait_ld();
      float mx4[4];                                            // four independent chains
#pragma unroll
      for (int j = 0; j < 4; ++j) mx4[j] = fmaxf(__uint_as_float(s0[j]), __uint_as_float(s1[j]));
#pragma unroll
      for (int i = 4; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], fmaxf(__uint_as_float(s0[i]), __uint_as_float(s1[i])));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float corr = ex2(m_run - m_new);
      const float neg_m = -m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      // p = 2^(s*scale - m_new) as packed bf16, written over the first 32 columns of this S buffer
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float p0 = ex2(fmaf(__uint_as_float(s0[2 * j]), p.scale_log2, neg_m));
        const float p1 = ex2(fmaf(__uint_as_float(s0[2 * j + 1]), p.scale_log2, neg_m));
        sum4[j & 3] += p0 + p1;
        const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
        w[j] = *reinterpret_cast<const uint32_t*>(&pk);
      }
      tc_st16(t_row + (uint32_t)(sb * kBK), w);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float p0 = ex2(fmaf(__uint_as_float(s1[2 * j]), p.scale_log2, neg_m));
        const float p1 = ex2(fmaf(__uint_as_float(s1[2 * j + 1]), p.scale_log2, neg_m));
        sum4[j & 3] += p0 + p1;
        const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
        w[j] = *reinterpret_cast<const uint32_t*>(&pk);
      }
      tc_st16(t_row + (uint32_t)(sb * kBK + 16), w);
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_P_READY + sb));
      l_run = l_run * corr + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
      m_run = m_new;
      if (kb >= 1) {
        // fold the previous block's product in, one block late: o <- o * corr(kb-1) + PV(kb-1)
        ok = mbar_wait(bar(BAR_PV_READY), (kb - 1) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        tc_ld32(t_row + kColPV, s0);
        tc_ld32(t_row + kColPV + 32u, s1);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_PV_FREE));
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          o[i] = fmaf(o[i], corr_prev, __uint_as_float(s0[i]));
          o[32 + i] = fmaf(o[32 + i], corr_prev, __uint_as_float(s1[i]));
        }
      }
      corr_prev = corr;
    }
    if (ok) {
      ok = mbar_wait(bar(BAR_PV_READY), (n_blocks - 1) & 1, s_abort, sync);
      if (ok) {
        uint32_t s0[32], s1[32];
        tc_fence_after();
        tc_ld32(t_row + kColPV, s0);
        tc_ld32(t_row + kColPV + 32u, s1);
        tc_wait_ld();
        tc_fence_before();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          o[i] = fmaf(o[i], corr_prev, __uint_as_float(s0[i]));
          o[32 + i] = fmaf(o[32 + i], corr_prev, __uint_as_float(s1[i]));
        }
      }
    }
    if (ok && row_ok) {
      p.st_m[sidx * p.H + h] = m_run;
      p.st_l[sidx * p.H + h] = l_run;
      float4* dst = reinterpret_cast<float4*>(p.st_o + sidx * p.d + h * kHeadDim);
#pragma unroll
      for (int i = 0; i < kHeadDim / 4; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------ host

// [rows, B, H, 64] bf16 viewed as a 4-D tensor; a box is `box_rows` rows of one head of one sequence.
static bool make_map(CUtensorMap* map, const void* base, int rows, int B, int H, int box_rows) {
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

// rows_q / rows_kv: number of rows the query buffer / caches hold (bounds for the tensor maps).
cudaError_t tile_tc_launch(const TileParams& p, int rows_q, int rows_kv, SyncArea* sync, cudaStream_t s) {
  const int nq = p.q1 - p.q0;
  if (nq <= 0 || p.k1 <= p.k0) return cudaSuccess;
  (void)rows_q;
  CUtensorMap mk, mv;
  if (!make_map(&mk, p.k_cache, rows_kv, p.B, p.H, kBK) || !make_map(&mv, p.v_cache, rows_kv, p.B, p.H, kBK))
    return cudaErrorInvalidValue;
  const size_t smem = TcSmem::total + 1024;
  cudaError_t e = cudaFuncSetAttribute(tile_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(ceil_div(nq, kBM), p.B * p.H);
  tile_tc_kernel<<<grid, kTcThreads, smem, s>>>(mk, mv, p, sync);
  return cudaGetLastError();
}

}  // namespace rt
