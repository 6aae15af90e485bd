// Parallel sweep over all positions at once (Sec. 6, activation checkpointing): with the layer
// outputs z known, every persistent pair can be rebuilt at once (Eqs. 1-2) and every a_i, z_i
// recomputed independently of the others.  The position-wise part of that sweep is a chain of dense
// products over all B*N rows, which is what this file holds:
//   c   = o / l                                 (attention value per head from the running stats)
//   h   = x + alpha W_o c                       (first display of Sec. 2.2)
//   u   = RMS_{g_mlp}(h)
//   g   = GELU(W_up u)
//   z'  = h + alpha W_down g
// Rows are position-major (m = position * B + sequence) as everywhere in the workspace.
// bf16 storage with column counts that are multiples of 128 takes the tcgen05 kernel (same main loop
// as the pre-pass projection: TMA ring of 64-wide K blocks, 128 x 128 accumulator in TMEM, one output
// row per epilogue thread); everything else takes a plain SIMT product.
#include "rt_kernels.h"
#include "rt_tc.cuh"

namespace rt {

__device__ __forceinline__ float gelu_exact(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)); }

// ---- c = o / l ------------------------------------------------------------------------------
template <typename T>
__global__ void attn_value_kernel(const float* st_o, const float* st_l, T* c, long long rows, int d, int H) {
  grid_dep_sync();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;       // one thread = 4 columns
  const long long total = rows * (d / 4);
  if (i >= total) return;
  const long long m = i / (d / 4);
  const int col = (int)(i % (d / 4)) * 4;
  const float il = 1.0f / st_l[m * H + col / kHeadDim];
  const float4 o = *reinterpret_cast<const float4*>(st_o + m * d + col);
  T* dst = c + m * d + col;
  dst[0] = from_f<T>(o.x * il); dst[1] = from_f<T>(o.y * il); dst[2] = from_f<T>(o.z * il); dst[3] = from_f<T>(o.w * il);
}

// ---- u = RMS_g(h) for fp32 rows -------------------------------------------------------------------
template <typename T>
__global__ void rms_rows_f32_kernel(const float* h, const T* g, T* u, int rows, int d, float eps, int pre) {
  grid_dep_sync();
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (m >= rows) return;
  const float* hr = h + (size_t)m * d;
  float ss = 0.f;
  for (int k = lane; k < d; k += 32) ss += hr[k] * hr[k];
  ss = warp_sum(ss);
  const float rs = pre ? rsqrtf(ss / (float)d + eps) : 1.0f;
  for (int k = lane; k < d; k += 32) u[(size_t)m * d + k] = from_f<T>(hr[k] * rs * (pre ? gain_at(g, k) : 1.0f));
}

// ---- epilogues of the dense products ------------------------------------------------------------
// value(m, n, acc) -> stored where the epilogue says; m = r * B + b
template <typename T>
__device__ __forceinline__ void epi_store(const DenseParams& p, int m, int n, float acc) {
  if (p.epi == DENSE_RES_X) {                                  // h = x + alpha acc  (fp32, position-major)
    const int b = m % p.B, r = m / p.B;
    const float xv = to_f(reinterpret_cast<const T*>(p.x)[(size_t)b * p.x_bs + (size_t)r * p.x_ts + n]);
    p.h[(size_t)m * p.N + n] = xv + p.alpha * acc;
  } else if (p.epi == DENSE_GELU) {                            // g = GELU(acc)  (storage type)
    reinterpret_cast<T*>(p.out)[(size_t)m * p.N + n] = from_f<T>(gelu_exact(acc));
  } else if (p.epi == DENSE_F32) {                             // C itself (fp32 [M, N]), optionally added to what is there
    float* dst = p.h + (size_t)m * p.N + n;
    *dst = (p.accumulate ? *dst : 0.f) + p.alpha * acc;
  } else {                                                     // z' = h + alpha acc  (storage type, caller's strides)
    const int b = m % p.B, r = m / p.B;
    reinterpret_cast<T*>(p.out)[(size_t)b * p.o_bs + (size_t)r * p.o_ts + n] = from_f<T>(p.h[(size_t)m * p.N + n] + p.alpha * acc);
  }
}

// ---- SIMT product: C[m, n] = sum_k A[m,k] W[n,k] ----------------------------------------------------
constexpr int kDM = 64, kDN = 64, kDK = 16;

template <typename T>
__global__ void __launch_bounds__(256) dense_simt_kernel(const DenseParams p) {
  __shared__ float As[kDK][kDM + 4];
  __shared__ float Bs[kDK][kDN + 4];
  const T* A = reinterpret_cast<const T*>(p.A);
  const T* W = reinterpret_cast<const T*>(p.W);
  const int m0 = blockIdx.x * kDM, n0 = blockIdx.y * kDN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const int lr = tid >> 2, lk = (tid & 3) * 4;
  for (int k0 = 0; k0 < p.K; k0 += kDK) {
    float f[4] = {0.f, 0.f, 0.f, 0.f}, g[4] = {0.f, 0.f, 0.f, 0.f};
    if (m0 + lr < p.M) reinterpret_cast<const Vec4<T>*>(A + (size_t)(m0 + lr) * p.K + k0 + lk)->to_float(f);
    if (n0 + lr < p.N) reinterpret_cast<const Vec4<T>*>(W + (size_t)(n0 + lr) * p.K + k0 + lk)->to_float(g);
#pragma unroll
    for (int i = 0; i < 4; ++i) { As[lk + i][lr] = f[i]; Bs[lk + i][lr] = g[i]; }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kDK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < p.N) epi_store<T>(p, m, n, acc[i][j]);
    }
  }
}

// ---- tcgen05 product (bf16; N a multiple of 128, K a multiple of 64) ------------------------------------
// Output tile 128 x BN.  BN = 256 halves the bytes fetched from L2 per product (the 128 x 128 tile is bound by the
// L2 -> SM stream: 32 KB per 2 MFLOP); its two 48 KB stages still leave room for two CTAs per SM.
constexpr int kTBK = 64, kTThreads = 192;
constexpr uint32_t kTABytes = kBM * kTBK * 2;

template <int BN>
struct DenseSmem {
  static constexpr int stages = BN == 256 ? 2 : 3;
  static constexpr uint32_t b_bytes = BN * kTBK * 2;
  static constexpr uint32_t a = 0;
  static constexpr uint32_t b = a + stages * kTABytes;
  static constexpr uint32_t bars = b + stages * b_bytes;         // full[], empty[], acc_ready
  static constexpr uint32_t tmem_ptr = bars + 64;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};

// Epilogue of one thread's output row: its BN accumulator columns from TMEM (lane = row), 32 at a time.
template <int BN>
__device__ __forceinline__ void dense_epilogue_row(const DenseParams& p, uint32_t tmem, int warp, int m, int n0, int splits, int zsplit) {
  const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
  const int b = m % p.B, r = m / p.B;
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    uint32_t v[32];
    tc_ld32(t_row + (uint32_t)c0, v);
    tc_wait_ld();
    if (m >= p.M) continue;
    const int n = n0 + c0;
    if (splits > 1) {                                          // raw partial sums; dense_reduce_kernel finishes
      float4* dst = reinterpret_cast<float4*>(p.partial + ((size_t)zsplit * p.M + m) * p.N + n);
#pragma unroll
      for (int q = 0; q < 8; ++q)
        dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
      continue;
    }
    if (p.epi == DENSE_F32) {
      float4* dst = reinterpret_cast<float4*>(p.h + (size_t)m * p.N + n);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 o = make_float4(p.alpha * __uint_as_float(v[4 * q]), p.alpha * __uint_as_float(v[4 * q + 1]),
                               p.alpha * __uint_as_float(v[4 * q + 2]), p.alpha * __uint_as_float(v[4 * q + 3]));
        if (p.accumulate) { const float4 old = dst[q]; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
        dst[q] = o;
      }
      continue;
    }
    if (p.epi == DENSE_RES_X) {
      const uint4* xs = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.x) + (size_t)b * p.x_bs + (size_t)r * p.x_ts + n);
      float4* dst = reinterpret_cast<float4*>(p.h + (size_t)m * p.N + n);
#pragma unroll
      for (int q = 0; q < 4; ++q) {                           // 8 columns per 16-byte load of x
        const uint4 xw = xs[q];
        const unsigned w4[4] = {xw.x, xw.y, xw.z, xw.w};
        float o[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          o[2 * j] = __uint_as_float(w4[j] << 16) + p.alpha * __uint_as_float(v[8 * q + 2 * j]);
          o[2 * j + 1] = __uint_as_float(w4[j] & 0xffff0000u) + p.alpha * __uint_as_float(v[8 * q + 2 * j + 1]);
        }
        dst[2 * q] = make_float4(o[0], o[1], o[2], o[3]);
        dst[2 * q + 1] = make_float4(o[4], o[5], o[6], o[7]);
      }
    } else {
      float o[32];
      if (p.epi == DENSE_GELU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = gelu_exact(__uint_as_float(v[j]));
      } else {
        const float4* hs = reinterpret_cast<const float4*>(p.h + (size_t)m * p.N + n);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 hv = hs[q];
          o[4 * q] = hv.x + p.alpha * __uint_as_float(v[4 * q]);
          o[4 * q + 1] = hv.y + p.alpha * __uint_as_float(v[4 * q + 1]);
          o[4 * q + 2] = hv.z + p.alpha * __uint_as_float(v[4 * q + 2]);
          o[4 * q + 3] = hv.w + p.alpha * __uint_as_float(v[4 * q + 3]);
        }
      }
      __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(p.out) +
                          (p.epi == DENSE_GELU ? (size_t)m * p.N + n : (size_t)b * p.o_bs + (size_t)r * p.o_ts + n);
      uint4* dst = reinterpret_cast<uint4*>(ob);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat162 pk = __floats2bfloat162_rn(o[8 * q + 2 * j], o[8 * q + 2 * j + 1]);
          w[j] = *reinterpret_cast<const uint32_t*>(&pk);
        }
        dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
}

template <int BN>
__global__ void __launch_bounds__(kTThreads, 2)
dense_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const DenseParams p,
                SyncArea* sync) {
  grid_dep_sync();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  using DS = DenseSmem<BN>;
  constexpr int kTStages = DS::stages;
  constexpr int kTBN = BN;
  constexpr uint32_t kTBBytes = DS::b_bytes;
  const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * kTBN;
  // split z of the contraction: k blocks [kb0, kb0 + n_kb)
  const int splits = p.splits > 1 ? p.splits : 1;
  const int kb_all = p.K / kTBK;
  const int kb0 = (int)((long long)kb_all * blockIdx.z / splits);
  const int n_kb = (int)((long long)kb_all * (blockIdx.z + 1) / splits) - kb0;
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + DS::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + DS::tmem_ptr);
  auto full = [&](int s) { return sbase + DS::bars + 8u * (uint32_t)s; };
  auto empty = [&](int s) { return sbase + DS::bars + 8u * (uint32_t)(kTStages + s); };
  const uint32_t acc_ready = sbase + DS::bars + 8u * (2 * kTStages);

  if (tid == 0) {
    *s_abort = 0;
    for (int s = 0; s < kTStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(acc_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + DS::tmem_ptr), "n"(kTBN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kTStages;
        if (kb >= kTStages) ok = mbar_wait(empty(s), ((kb / kTStages) - 1) & 1, s_abort, sync);
        if (!ok) break;
        mbar_expect_tx(full(s), kTABytes + kTBBytes);
        tma_load_2d(sbase + DS::a + s * kTABytes, &map_a, full(s), (kb0 + kb) * kTBK, m0);
        tma_load_2d(sbase + DS::b + s * kTBBytes, &map_w, full(s), (kb0 + kb) * kTBK, n0);
        ++issued;
      }
      if (!ok) {
        // gave up: let the copies already started land before the shared memory goes away (bounded)
        for (int i = issued > kTStages ? issued - kTStages : 0; i < issued; ++i) {
          unsigned spins = 0;
          while (!mbar_try_wait(full(i % kTStages), (i / kTStages) & 1) && ++spins < (1u << 20)) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kTBN, false);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kTStages;
        ok = mbar_wait(full(s), (kb / kTStages) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a0 = make_desc(sbase + DS::a + s * kTABytes, 16, 1024);
        const uint64_t b0 = make_desc(sbase + DS::b + s * kTBBytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kTBK / 16; ++ks)
          tc_mma(tmem, a0 + 2u * ks, b0 + 2u * ks, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
        tc_commit(empty(s));
      }
      if (ok) tc_commit(acc_ready);
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: one output row per thread, 32 columns at a time ----------------
    const int m = m0 + warp * 32 + lane;
    if (mbar_wait(acc_ready, 0, s_abort, sync)) {
      tc_fence_after();
      dense_epilogue_row<kTBN>(p, tmem, warp, m, n0, splits, (int)blockIdx.z);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTBN) : "memory");
  }
}

// ---- the same product on CTA pairs (cta_group::2) -----------------------------------------------------------
// Two CTAs of a cluster share a 256 x BN output tile: each fetches its own 128 rows of A and HALF of the BN weight rows,
// the leader's thread issues tcgen05.mma.cta_group::2 (M = 256), which reads A and W from both CTAs' shared memory and
// accumulates each CTA's 128 rows in that CTA's TMEM.  Per CTA and 64-wide k-block that is 16 KB + BN * 64 bytes from L2
// instead of 16 KB + BN * 128: the products here are bound by that stream.  Copies are plain TMA loads, one per CTA,
// that report to the leader's barrier; the leader's commits arrive on both CTAs' barriers.
template <int BN>
struct PairSmem {
  static constexpr int stages = BN == 256 ? 3 : 4;
  static constexpr uint32_t b_bytes = (BN / 2) * kTBK * 2;
  static constexpr uint32_t a = 0;
  static constexpr uint32_t b = a + stages * kTABytes;
  static constexpr uint32_t bars = b + stages * b_bytes;         // full[], empty[], acc_ready
  static constexpr uint32_t tmem_ptr = bars + 128;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of this CTA's tile whose bytes are reported to the LEADER's barrier at the same offset (bit 24 of a
// shared::cluster address selects the CTA of the pair)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar & 0xFEFFFFFFu), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Issued by the leader: arrives on the barrier at this offset in BOTH CTAs once the pair's products so far are done
// (one commit per CTA's barrier; the partner's address comes from mapa).
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  uint32_t peer;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(peer) : "r"(bar), "r"(1u));
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(peer) : "memory");
}

template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTThreads, 2)
dense_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const DenseParams p,
                  SyncArea* sync) {
  grid_dep_sync();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  using PS = PairSmem<BN>;
  constexpr int kSt = PS::stages;
  const int rank = (int)cluster_rank();                         // 0: leader (issues the products)
  const int m0 = ((int)blockIdx.x >> 1) * 2 * kBM + rank * kBM, n0 = blockIdx.y * BN;
  const int splits = p.splits > 1 ? p.splits : 1;
  const int kb_all = p.K / kTBK;
  const int kb0 = (int)((long long)kb_all * blockIdx.z / splits);
  const int n_kb = (int)((long long)kb_all * (blockIdx.z + 1) / splits) - kb0;
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + PS::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + PS::tmem_ptr);
  auto full = [&](int s) { return sbase + PS::bars + 8u * (uint32_t)s; };
  auto empty = [&](int s) { return sbase + PS::bars + 8u * (uint32_t)(kSt + s); };
  const uint32_t acc_ready = sbase + PS::bars + 8u * (2 * kSt);

  if (tid == 0) {
    *s_abort = 0;
    for (int s = 0; s < kSt; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(acc_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + PS::tmem_ptr), "n"(BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                           // both CTAs' barriers exist before anything is signalled
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // No role returns early: every thread of both CTAs reaches the cluster barrier at the end.
  if (warp == 4) {
    // ---------------- TMA producer (each CTA: its 128 rows of A, its half of the weight rows) ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kSt;
        if (kb >= kSt) ok = mbar_wait(empty(s), ((kb / kSt) - 1) & 1, s_abort, sync);
        if (!ok) break;
        if (rank == 0) mbar_expect_tx(full(s), 2u * (kTABytes + PS::b_bytes));      // the bytes of both CTAs
        tma_load_2d_pair(sbase + PS::a + s * kTABytes, &map_a, full(s), (kb0 + kb) * kTBK, m0);
        tma_load_2d_pair(sbase + PS::b + s * PS::b_bytes, &map_w, full(s), (kb0 + kb) * kTBK, n0 + rank * (BN / 2));
        ++issued;
      }
      (void)issued;
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------- MMA issuer (leader only) ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kSt;
        ok = mbar_wait(full(s), (kb / kSt) & 1, s_abort, sync);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a0 = make_desc(sbase + PS::a + s * kTABytes, 16, 1024);
        const uint64_t b0 = make_desc(sbase + PS::b + s * PS::b_bytes, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < kTBK / 16; ++ks)
          tc_mma_pair(tmem, a0 + 2u * ks, b0 + 2u * ks, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
        tc_commit_pair(empty(s));
      }
      if (ok) tc_commit_pair(acc_ready);
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: one output row per thread ----------------
    const int m = m0 + warp * 32 + lane;
    if (mbar_wait(acc_ready, 0, s_abort, sync)) {
      tc_fence_after();
      dense_epilogue_row<BN>(p, tmem, warp, m, n0, splits, (int)blockIdx.z);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                           // the partner is done with this CTA's shared memory and TMEM
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(BN) : "memory");
  }
}

// ---- CTA pairs, persistent: one pair per two SMs walks over the 256 x 256 output tiles ----------------------------
// Same products as dense_pair_kernel, but a pair stays resident (one CTA per SM, all 512 TMEM columns = two accumulator
// buffers of 256) and takes tile after tile: while the epilogue warps of both CTAs drain buffer b, the leader already
// accumulates the next tile into buffer b ^ 1, and the operand ring never runs dry between tiles.
struct PersistSmem {
  static constexpr int stages = 6;
  static constexpr uint32_t b_bytes = 128 * kTBK * 2;            // half of a 256-column weight tile
  static constexpr uint32_t a = 0;
  static constexpr uint32_t b = a + stages * kTABytes;
  static constexpr uint32_t bars = b + stages * b_bytes;         // full[6], empty[6], acc_full[2], acc_empty[2]
  static constexpr uint32_t tmem_ptr = bars + 192;
  static constexpr uint32_t abort_flag = tmem_ptr + 8;
  static constexpr uint32_t total = abort_flag + 8;
};
// arrive on the barrier at this offset in the LEADER's shared memory (from either CTA of the pair)
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(bar), "r"(0u));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}

// One thread's row of a q / k~ / v~ tile: 64 columns (one head) at a time, qkRMS over the head for q and k, bf16 out.
__device__ __forceinline__ void qkv_epilogue_row(const DenseParams& p, uint32_t tmem, int warp, int m, int which, int col0) {
  const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
  const bool qkn = p.qk_norm != 0 && which < 2;
  const __nv_bfloat16* gain = reinterpret_cast<const __nv_bfloat16*>(which == 0 ? p.g_q : p.g_k);
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(which == 0 ? p.q_out : (which == 1 ? p.k_out : p.v_out));
#pragma unroll 1
  for (int hh = 0; hh < 256 / kHeadDim; ++hh) {
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
      rs = rsqrtf(ss * (1.0f / kHeadDim) + p.qk_eps);
    }
    if (m >= p.M) continue;
    const int c_head = col0 + hh * kHeadDim;
    uint4* dst = reinterpret_cast<uint4*>(out + (size_t)m * p.N + c_head);
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {                           // 8 columns = 16 bytes per store
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

// QKV: the three projections of the pre-pass (p.epi == DENSE_QKV; tiles walk over q, then k~, then v~ columns, each
// with its own weight map); otherwise one product with map_w (map_w2, map_w3 unused).
template <bool QKV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTThreads, 1)
dense_pair_persist_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                          const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_w3, const DenseParams p,
                          SyncArea* sync) {
  grid_dep_sync();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  using PS = PersistSmem;
  constexpr int kSt = PS::stages, BN = 256;
  const int rank = (int)cluster_rank();
  const int m_pairs = (p.M + 2 * kBM - 1) / (2 * kBM), n_per_mat = p.N / BN, n_tiles = (QKV ? 3 : 1) * n_per_mat;
  const int T = m_pairs * n_tiles;                              // tiles; pair c takes c, c + pairs, ...
  const int pairs = (int)gridDim.x >> 1, pair_id = (int)blockIdx.x >> 1;
  const int n_kb = p.K / kTBK;
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + PS::abort_flag);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + PS::tmem_ptr);
  auto full = [&](int s) { return sbase + PS::bars + 8u * (uint32_t)s; };
  auto empty = [&](int s) { return sbase + PS::bars + 8u * (uint32_t)(kSt + s); };
  auto acc_full = [&](int b) { return sbase + PS::bars + 8u * (uint32_t)(2 * kSt + b); };
  auto acc_empty = [&](int b) { return sbase + PS::bars + 8u * (uint32_t)(2 * kSt + 2 + b); };

  if (tid == 0) {
    *s_abort = 0;
    for (int s = 0; s < kSt; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 8); }   // 4 epilogue warps of each CTA
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + PS::tmem_ptr), "n"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // No role returns early: every thread of both CTAs reaches the cluster barrier at the end.
  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (int t = pair_id; t < T && ok; t += pairs) {
        const int nt = t / m_pairs, which = QKV ? nt / n_per_mat : 0;
        const int m0 = (t % m_pairs) * 2 * kBM + rank * kBM, n0 = (QKV ? nt % n_per_mat : nt) * BN;
        const CUtensorMap* mw = which == 0 ? &map_w : (which == 1 ? &map_w2 : &map_w3);
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % kSt;
          if (it >= kSt) ok = mbar_wait(empty(s), ((it / kSt) - 1) & 1, s_abort, sync);
          if (!ok) break;
          if (rank == 0) mbar_expect_tx(full(s), 2u * (kTABytes + PS::b_bytes));
          tma_load_2d_pair(sbase + PS::a + s * kTABytes, &map_a, full(s), kb * kTBK, m0);
          tma_load_2d_pair(sbase + PS::b + s * PS::b_bytes, mw, full(s), kb * kTBK, n0 + rank * (BN / 2));
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------- MMA issuer (leader only) ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24);
      int it = 0, i = 0;
      bool ok = true;
      for (int t = pair_id; t < T && ok; t += pairs, ++i) {
        const int b = i & 1;
        if (i >= 2) ok = mbar_wait(acc_empty(b), ((i >> 1) - 1) & 1, s_abort, sync);     // both CTAs have drained this buffer
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % kSt;
          ok = mbar_wait(full(s), (it / kSt) & 1, s_abort, sync);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a0 = make_desc(sbase + PS::a + s * kTABytes, 16, 1024);
          const uint64_t b0 = make_desc(sbase + PS::b + s * PS::b_bytes, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < kTBK / 16; ++ks)
            tc_mma_pair(tmem + (uint32_t)(b * BN), a0 + 2u * ks, b0 + 2u * ks, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
          tc_commit_pair(empty(s));
        }
        if (ok) tc_commit_pair(acc_full(b));
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: one output row per thread, tile after tile ----------------
    int i = 0;
    bool ok = true;
    for (int t = pair_id; t < T && ok; t += pairs, ++i) {
      const int b = i & 1;
      const int nt = t / m_pairs, which = QKV ? nt / n_per_mat : 0;
      const int m = (t % m_pairs) * 2 * kBM + rank * kBM + warp * 32 + lane, n0 = (QKV ? nt % n_per_mat : nt) * BN;
      ok = __all_sync(0xffffffffu, mbar_wait(acc_full(b), (i >> 1) & 1, s_abort, sync));
      if (!ok) break;
      tc_fence_after();
      if (QKV) qkv_epilogue_row(p, tmem + (uint32_t)(b * BN), warp, m, which, n0);
      else dense_epilogue_row<BN>(p, tmem + (uint32_t)(b * BN), warp, m, n0, 1, 0);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(acc_empty(b));
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(512) : "memory");
  }
}

// Sums the partial products of a split contraction in a fixed order and applies the epilogue; one CTA per
// output row, so it can also leave RMS_g(row) of the result for the product that follows.
template <typename T>
__global__ void __launch_bounds__(256) dense_reduce_kernel(const DenseParams p) {
  grid_dep_sync();
  __shared__ float red[8];
  const int m = blockIdx.x, tid = threadIdx.x;
  const int b = m % p.B, r = m / p.B;
  const T* g = reinterpret_cast<const T*>(p.norm_gain);
  if (p.N % 4 == 0 && p.N <= 4096) {
    // rows of up to 4096 entries: a thread owns up to four groups of four consecutive columns, fetched as 16-byte
    // loads (all of a thread's loads are independent) and kept in registers for the normalisation
    float v[4][4];
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int n = 4 * (tid + 256 * c);
      if (n >= p.N) break;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int z = 0; z < p.splits; ++z) {
        const float4 a = *reinterpret_cast<const float4*>(p.partial + ((size_t)z * p.M + m) * p.N + n);
        acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
      }
      const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
      if (p.epi == DENSE_RES_X) {
        const T* xs = reinterpret_cast<const T*>(p.x) + (size_t)b * p.x_bs + (size_t)r * p.x_ts + n;
#pragma unroll
        for (int j = 0; j < 4; ++j) v[c][j] = to_f(xs[j]) + p.alpha * a4[j];
        *reinterpret_cast<float4*>(p.h + (size_t)m * p.N + n) = make_float4(v[c][0], v[c][1], v[c][2], v[c][3]);
      } else if (p.epi == DENSE_GELU) {
        T* o = reinterpret_cast<T*>(p.out) + (size_t)m * p.N + n;
#pragma unroll
        for (int j = 0; j < 4; ++j) { v[c][j] = gelu_exact(a4[j]); o[j] = from_f<T>(v[c][j]); }
      } else if (p.epi == DENSE_F32) {
        float4* dst = reinterpret_cast<float4*>(p.h + (size_t)m * p.N + n);
        const float4 old = p.accumulate ? *dst : make_float4(0.f, 0.f, 0.f, 0.f);
        v[c][0] = old.x + p.alpha * a4[0]; v[c][1] = old.y + p.alpha * a4[1];
        v[c][2] = old.z + p.alpha * a4[2]; v[c][3] = old.w + p.alpha * a4[3];
        *dst = make_float4(v[c][0], v[c][1], v[c][2], v[c][3]);
      } else {
        const float4 hv = *reinterpret_cast<const float4*>(p.h + (size_t)m * p.N + n);
        const float h4[4] = {hv.x, hv.y, hv.z, hv.w};
        T* o = reinterpret_cast<T*>(p.out) + (size_t)b * p.o_bs + (size_t)r * p.o_ts + n;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const T zr = from_f<T>(h4[j] + p.alpha * a4[j]);
          o[j] = zr;
          v[c][j] = to_f(zr);                                  // the next product sees the stored (rounded) z
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) ss += v[c][j] * v[c][j];
    }
    if (!p.norm_out) return;
    ss = warp_sum(ss);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float rs = p.norm_pre ? rsqrtf(tot / (float)p.N + p.norm_eps) : 1.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int n = 4 * (tid + 256 * c);
      if (n >= p.N) break;
      T* o = reinterpret_cast<T*>(p.norm_out) + (size_t)m * p.N + n;
#pragma unroll
      for (int j = 0; j < 4; ++j) o[j] = from_f<T>(v[c][j] * rs * (p.norm_pre ? gain_at(g, n + j) : 1.0f));
    }
    return;
  }
  float ss = 0.f;
  for (int n = tid; n < p.N; n += 256) {
    float acc = 0.f;
    for (int z = 0; z < p.splits; ++z) acc += p.partial[((size_t)z * p.M + m) * p.N + n];
    float v;
    if (p.epi == DENSE_RES_X) {
      v = to_f(reinterpret_cast<const T*>(p.x)[(size_t)b * p.x_bs + (size_t)r * p.x_ts + n]) + p.alpha * acc;
      p.h[(size_t)m * p.N + n] = v;
    } else if (p.epi == DENSE_GELU) {
      v = gelu_exact(acc);
      reinterpret_cast<T*>(p.out)[(size_t)m * p.N + n] = from_f<T>(v);
    } else if (p.epi == DENSE_F32) {
      float* dst = p.h + (size_t)m * p.N + n;
      v = (p.accumulate ? *dst : 0.f) + p.alpha * acc;
      *dst = v;
    } else {
      const T zr = from_f<T>(p.h[(size_t)m * p.N + n] + p.alpha * acc);
      reinterpret_cast<T*>(p.out)[(size_t)b * p.o_bs + (size_t)r * p.o_ts + n] = zr;
      v = to_f(zr);                                              // the next product sees the stored (rounded) z
    }
    ss += v * v;
  }
  if (!p.norm_out) return;
  ss = warp_sum(ss);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float rs = p.norm_pre ? rsqrtf(tot / (float)p.N + p.norm_eps) : 1.0f;
  for (int n = tid; n < p.N; n += 256) {
    float v;
    if (p.epi == DENSE_RES_X) v = p.h[(size_t)m * p.N + n];
    else if (p.epi == DENSE_GELU) v = to_f(reinterpret_cast<const T*>(p.out)[(size_t)m * p.N + n]);
    else v = to_f(reinterpret_cast<const T*>(p.out)[(size_t)b * p.o_bs + (size_t)r * p.o_ts + n]);
    reinterpret_cast<T*>(p.norm_out)[(size_t)m * p.N + n] = from_f<T>(v * rs * (p.norm_pre ? gain_at(g, n + 0) : 1.0f));
  }
}

static_assert(kTBK == 64, "tensor_map_rows_bf16 encodes 64-column boxes");

cudaError_t dense_launch(int dtype, const DenseParams& p, SyncArea* sync, cudaStream_t s, bool* normed) {
  if (normed) *normed = false;
  if (p.M <= 0) return cudaSuccess;
  const bool strides_ok = p.epi == DENSE_GELU || p.epi == DENSE_F32 || (((p.epi == DENSE_RES_X ? p.x_bs : p.o_bs) % 8 == 0) &&
                                                  ((p.epi == DENSE_RES_X ? p.x_ts : p.o_ts) % 8 == 0));
  if (dtype == RT_BF16 && p.N % 128 == 0 && p.K % kTBK == 0 && strides_ok) {
    // Few rows (the wide-batch token step: M = B): narrow tiles and a split contraction so that the launch still
    // fills the GPU; the partial sums are combined in a fixed order by a second small kernel.
    const int sms = sm_count();
    const int m_tiles = ceil_div(p.M, kBM);
    int bn = p.N % 256 == 0 ? 256 : 128;
    if (bn == 256 && m_tiles * (p.N / 256) < sms) bn = 128;
    DenseParams q = p;
    q.splits = 1;
    const int ctas = m_tiles * (p.N / bn), kb_all = p.K / kTBK;
    if (p.partial && ctas < sms / 2 && kb_all >= 8) {
      int want = (sms + ctas - 1) / ctas;                         // about one wave
      if (want > 8) want = 8;
      while (want > 1 && kb_all / want < 4) --want;               // at least 4 k blocks per split
      if ((size_t)want * p.M * p.N * sizeof(float) <= p.partial_bytes) q.splits = want;
    }
    // CTA pairs on 256-row tiles (each CTA fetches half of the weight tile) for products of at least a wave of CTAs:
    // c3's chain products 0.892 -> 0.850 ms; the few-row products of a wide-batch token step are 3 % slower as pairs
    const bool pair = q.splits == 1 && ctas >= sms;
    CUtensorMap ma, mw;
    if (!tensor_map_rows_bf16(&ma, p.A, p.M, p.K, kBM) || !tensor_map_rows_bf16(&mw, p.W, p.N, p.K, pair ? bn / 2 : bn)) return cudaErrorInvalidValue;
    dim3 grid(pair ? 2 * ceil_div(p.M, 2 * kBM) : m_tiles, p.N / bn, q.splits);
    auto run = [&](auto kern, size_t smem) -> cudaError_t {
      cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), (int)smem);
      if (e != cudaSuccess) return e;
      return launch_chained(kern, grid, dim3(kTThreads), smem, s, p.chained != 0, ma, mw, q, sync);
    };
    cudaError_t e;
#ifndef RT_DENSE_PERSIST
#define RT_DENSE_PERSIST 1
#endif
    if (pair && bn == 256 && RT_DENSE_PERSIST) {
      // resident pairs (one CTA per SM) walking over the tiles, two accumulator buffers
      const int tiles = ceil_div(p.M, 2 * kBM) * (p.N / 256), max_pairs = sms / 2;
      grid = dim3(2 * (tiles < max_pairs ? tiles : max_pairs), 1, 1);
      e = ensure_dynamic_smem(reinterpret_cast<const void*>(&dense_pair_persist_kernel<false>), (int)(PersistSmem::total + 1024));
      if (e == cudaSuccess)
        e = launch_chained(dense_pair_persist_kernel<false>, grid, dim3(kTThreads), PersistSmem::total + 1024, s, p.chained != 0, ma, mw, mw, mw, q, sync);
    } else if (pair) e = bn == 256 ? run(dense_pair_kernel<256>, PairSmem<256>::total + 1024) : run(dense_pair_kernel<128>, PairSmem<128>::total + 1024);
    else e = bn == 256 ? run(dense_tc_kernel<256>, DenseSmem<256>::total + 1024) : run(dense_tc_kernel<128>, DenseSmem<128>::total + 1024);
    if (e != cudaSuccess) return e;
    if (q.splits > 1) {
      cudaError_t er = launch_chained(dense_reduce_kernel<__nv_bfloat16>, dim3(p.M), dim3(256), 0, s, p.chained != 0, q);
      if (er != cudaSuccess) return er;
      if (normed && p.norm_out) *normed = true;
    }
    return cudaGetLastError();
  }
  dim3 grid(ceil_div(p.M, kDM), ceil_div(p.N, kDN));
  if (dtype == RT_BF16) dense_simt_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(p);
  else dense_simt_kernel<float><<<grid, 256, 0, s>>>(p);
  return cudaGetLastError();
}

bool dense_qkv_pair_supported(int M, int d) {
  return d % 256 == 0 && ceil_div(M, 2 * kBM) * 3 * (d / 256) >= sm_count() / 2;
}

cudaError_t dense_qkv_pair_launch(const DenseParams& p, SyncArea* sync, cudaStream_t s) {
  CUtensorMap ma, m1, m2, m3;
  if (!tensor_map_rows_bf16(&ma, p.A, p.M, p.K, kBM) || !tensor_map_rows_bf16(&m1, p.W, p.N, p.K, 128) ||
      !tensor_map_rows_bf16(&m2, p.W2, p.N, p.K, 128) || !tensor_map_rows_bf16(&m3, p.W3, p.N, p.K, 128))
    return cudaErrorInvalidValue;
  const int tiles = ceil_div(p.M, 2 * kBM) * 3 * (p.N / 256), max_pairs = sm_count() / 2;
  dim3 grid(2 * (tiles < max_pairs ? tiles : max_pairs), 1, 1);
  const size_t smem = PersistSmem::total + 1024;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&dense_pair_persist_kernel<true>), (int)smem);
  if (e != cudaSuccess) return e;
  return launch_chained(dense_pair_persist_kernel<true>, grid, dim3(kTThreads), smem, s, p.chained != 0, ma, m1, m2, m3, p, sync);
}

cudaError_t attn_value_launch(int dtype, const float* st_o, const float* st_l, void* c, long long rows, int d, int H, cudaStream_t s,
                              bool chained) {
  const long long total = rows * (d / 4);
  const dim3 blocks((unsigned)((total + 255) / 256));
  if (dtype == RT_BF16) return launch_chained(attn_value_kernel<__nv_bfloat16>, blocks, dim3(256), 0, s, chained, st_o, st_l, (__nv_bfloat16*)c, rows, d, H);
  return launch_chained(attn_value_kernel<float>, blocks, dim3(256), 0, s, chained, st_o, st_l, (float*)c, rows, d, H);
}

cudaError_t rms_rows_f32_launch(int dtype, const float* h, const void* g, void* u, int rows, int d, float eps, int pre, cudaStream_t s,
                                bool chained) {
  const dim3 blocks(ceil_div(rows, 8));
  if (dtype == RT_BF16) return launch_chained(rms_rows_f32_kernel<__nv_bfloat16>, blocks, dim3(256), 0, s, chained, h, (const __nv_bfloat16*)g, (__nv_bfloat16*)u, rows, d, eps, pre);
  return launch_chained(rms_rows_f32_kernel<float>, blocks, dim3(256), 0, s, chained, h, (const float*)g, (float*)u, rows, d, eps, pre);
}

}  // namespace rt
