// Cross-block tile on the 5th-generation tensor cores (bf16 storage): Algorithm 2 (UpdateTile)
// for queries [q0,q1) against the revealed pairs [k0,k1), every sequence and head, with the
// running stats (m, l, o) carried in fp32 in the workspace.
//
// One CTA = 128 query rows of one (sequence, head) pair, looping over 64-key blocks:
//   TMA     Q tile once, K and V blocks double-buffered, straight out of the position-major
//           cache / query buffer (a 4-D tensor map picks the head's 64 columns of each row),
//           128-byte swizzle = the tensor cores' canonical shared-memory layout
//   S       tcgen05.mma  S[128x64] = Q[128x64] . K^T        (A, B K-major; accumulator in TMEM)
//   softmax 4 warps, one thread per query row: tcgen05.ld of the row, running max in log2 units,
//           p = 2^(s - m), row sum, P written to shared memory as bf16 in the swizzled layout
//   PV      tcgen05.mma  PV[128x64] = P[128x64] . V[64x64]  (B is MN-major: V rows are keys)
//   merge   o = o * 2^(m_old - m_new) + PV in registers (fp32), l likewise
// A fifth warp owns TMEM allocation, issues the TMA copies and (one elected lane) the MMAs.
// Three CTAs fit on an SM (64 KB shared memory, 128 TMEM columns each), so the softmax of one CTA
// overlaps the MMAs of the others.  Every mbarrier wait is bounded: on expiry the CTA records
// RT_ERR_TIMEOUT, stops issuing work, waits (bounded) for its copies in flight, frees its TMEM and
// returns.
#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

constexpr int kBK = 64;                // keys per block
constexpr int kTcThreads = 160;        // 4 softmax warps + 1 control warp
constexpr int kTmemCols = 128;         // S: columns [0,64), PV: columns [64,128)
constexpr uint32_t kQBytes = kBM * kHeadDim * 2;     // 16 KB
constexpr uint32_t kKVBytes = kBK * kHeadDim * 2;    // 8 KB
constexpr uint32_t kPBytes = kBM * kBK * 2;          // 16 KB

struct TcSmem {                        // offsets from a 1024-byte aligned base
  static constexpr uint32_t q = 0;
  static constexpr uint32_t k = q + kQBytes;                 // 2 stages
  static constexpr uint32_t v = k + 2 * kKVBytes;            // 2 stages
  static constexpr uint32_t p = v + 2 * kKVBytes;
  static constexpr uint32_t bars = p + kPBytes;              // 10 mbarriers
  static constexpr uint32_t tmem_ptr = bars + 128;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};
enum { BAR_Q = 0, BAR_KV_FULL = 1, BAR_KV_EMPTY = 3, BAR_S_READY = 5, BAR_S_FREE = 6, BAR_P_READY = 7,
       BAR_PV_READY = 8, BAR_PV_FREE = 9 };

__global__ void __launch_bounds__(kTcThreads, 3)
tile_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const TileParams p, SyncArea* sync) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  const int qb = p.q0 + blockIdx.x * kBM;                 // first query row of this CTA
  const int nk = p.k1 - p.k0;
  const int n_blocks = (nk + kBK - 1) / kBK;
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + TcSmem::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + TcSmem::tmem_ptr);
  auto bar = [&](int i) { return sbase + TcSmem::bars + 8u * (uint32_t)i; };

  if (tid == 0) {
    *s_abort = 0;
    mbar_init(bar(BAR_Q), 1);
    mbar_init(bar(BAR_KV_FULL), 1); mbar_init(bar(BAR_KV_FULL + 1), 1);
    mbar_init(bar(BAR_KV_EMPTY), 1); mbar_init(bar(BAR_KV_EMPTY + 1), 1);
    mbar_init(bar(BAR_S_READY), 1);
    mbar_init(bar(BAR_S_FREE), 4);
    mbar_init(bar(BAR_P_READY), 4);
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

  if (warp == 4) {
    // ------------------------------ control warp: TMA + MMA issue ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(kBK, false);
      constexpr uint32_t idesc_pv = make_idesc(kHeadDim, true);
      mbar_expect_tx(bar(BAR_Q), kQBytes);
      tma_load_4d(sbase + TcSmem::q, &map_q, bar(BAR_Q), 0, h, b, qb);
      mbar_expect_tx(bar(BAR_KV_FULL), 2 * kKVBytes);
      tma_load_4d(sbase + TcSmem::k, &map_k, bar(BAR_KV_FULL), 0, h, b, p.k0);
      tma_load_4d(sbase + TcSmem::v, &map_v, bar(BAR_KV_FULL), 0, h, b, p.k0);
      int loads_issued = 1;                                   // K/V blocks whose copies were started
      bool ok = mbar_wait(bar(BAR_Q), 0, s_abort, sync);
      for (int kb = 0; kb < n_blocks && ok; ++kb) {
        const int st = kb & 1;
        ok = mbar_wait(bar(BAR_KV_FULL + st), (kb >> 1) & 1, s_abort, sync);
        if (ok && kb > 0) ok = mbar_wait(bar(BAR_S_FREE), (kb - 1) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        {
          const uint64_t a0 = make_desc(sbase + TcSmem::q, 16, 1024);
          const uint64_t b0 = make_desc(sbase + TcSmem::k + st * kKVBytes, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < kHeadDim / 16; ++ks)          // 32 bytes along K per step
            tc_mma(tmem, a0 + 2u * ks, b0 + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
          tc_commit(bar(BAR_S_READY));
        }
        // next block's copies: its stage was last read by the PV product of block kb-1
        if (kb + 1 < n_blocks) {
          const int sn = (kb + 1) & 1;
          if (kb >= 1) ok = mbar_wait(bar(BAR_KV_EMPTY + sn), ((kb - 1) >> 1) & 1, s_abort, sync);
          if (!ok) break;
          mbar_expect_tx(bar(BAR_KV_FULL + sn), 2 * kKVBytes);
          tma_load_4d(sbase + TcSmem::k + sn * kKVBytes, &map_k, bar(BAR_KV_FULL + sn), 0, h, b, p.k0 + (kb + 1) * kBK);
          tma_load_4d(sbase + TcSmem::v + sn * kKVBytes, &map_v, bar(BAR_KV_FULL + sn), 0, h, b, p.k0 + (kb + 1) * kBK);
          ++loads_issued;
        }
        ok = mbar_wait(bar(BAR_P_READY), kb & 1, s_abort, sync);
        if (ok && kb > 0) ok = mbar_wait(bar(BAR_PV_FREE), (kb - 1) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        {
          const uint64_t a0 = make_desc(sbase + TcSmem::p, 16, 1024);
          const uint64_t b0 = make_desc(sbase + TcSmem::v + st * kKVBytes, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < kBK / 16; ++ks)               // A: 32 bytes along K; B (MN-major): 16 key rows = 2048 bytes
            tc_mma(tmem + 64u, a0 + 2u * ks, b0 + 128u * ks, idesc_pv, ks > 0 ? 1u : 0u);
          tc_commit(bar(BAR_PV_READY));
          tc_commit(bar(BAR_KV_EMPTY + st));
        }
      }
      if (!ok) {
        // gave up: let the copies already started land before the shared memory goes away (bounded)
        for (int i = 0; i < loads_issued && i < 2; ++i) {
          const int blk = loads_issued - 1 - i;
          unsigned spins = 0;
          while (!mbar_try_wait(bar(BAR_KV_FULL + (blk & 1)), (blk >> 1) & 1) && ++spins < (1u << 20)) {}
        }
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
    unsigned char* p_row = smem + TcSmem::p + (row >> 3) * 1024 + (row & 7) * 128;
    bool ok = true;
    for (int kb = 0; kb < n_blocks; ++kb) {
      const int n_valid = nk - kb * kBK < kBK ? nk - kb * kBK : kBK;
      ok = mbar_wait(bar(BAR_S_READY), kb & 1, s_abort, sync);
      if (!ok) break;
      tc_fence_after();
      uint32_t s0[32], s1[32];
      tc_ld32(t_row, s0);
      tc_ld32(t_row + 32u, s1);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_S_FREE));           // S may be overwritten by the next block's product
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        if (i < n_valid) mx = fmaxf(mx, __uint_as_float(s0[i]));
        if (32 + i < n_valid) mx = fmaxf(mx, __uint_as_float(s1[i]));
      }
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float corr = ex2(m_run - m_new);
      float sum = 0.f;
      // p = 2^(s*scale - m_new), packed to bf16 and stored in the swizzled K-major layout
#pragma unroll
      for (int c16 = 0; c16 < 8; ++c16) {                     // 16-byte chunk = 8 keys
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int e0 = c16 * 8 + 2 * j;
          const float x0 = __uint_as_float(e0 < 32 ? s0[e0 & 31] : s1[e0 & 31]);
          const float x1 = __uint_as_float(e0 + 1 < 32 ? s0[(e0 + 1) & 31] : s1[(e0 + 1) & 31]);
          const float p0 = e0 < n_valid ? ex2(fmaf(x0, p.scale_log2, -m_new)) : 0.f;
          const float p1 = e0 + 1 < n_valid ? ex2(fmaf(x1, p.scale_log2, -m_new)) : 0.f;
          const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
          // the row sum uses the rounded values the tensor core will see
          sum += __low2float(pk) + __high2float(pk);
          w[j] = *reinterpret_cast<const uint32_t*>(&pk);
        }
        *reinterpret_cast<uint4*>(p_row + ((c16 ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_P_READY));
      l_run = l_run * corr + sum;
      m_run = m_new;
      ok = mbar_wait(bar(BAR_PV_READY), kb & 1, s_abort, sync);
      if (!ok) break;
      tc_fence_after();
      tc_ld32(t_row + 64u, s0);
      tc_ld32(t_row + 96u, s1);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PV_FREE));
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        o[i] = fmaf(o[i], corr, __uint_as_float(s0[i]));
        o[32 + i] = fmaf(o[32 + i], corr, __uint_as_float(s1[i]));
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
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, p.q, rows_q, p.B, p.H, kBM) || !make_map(&mk, p.k_cache, rows_kv, p.B, p.H, kBK) ||
      !make_map(&mv, p.v_cache, rows_kv, p.B, p.H, kBK))
    return cudaErrorInvalidValue;
  const size_t smem = TcSmem::total + 1024;
  cudaError_t e = cudaFuncSetAttribute(tile_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(ceil_div(nq, kBM), p.B * p.H);
  tile_tc_kernel<<<grid, kTcThreads, smem, s>>>(mq, mk, mv, p, sync);
  return cudaGetLastError();
}

}  // namespace rt
