// Pre-pass of Algorithm 1: everything that depends only on the layer input and therefore
// runs for all positions at once (line 1: queries; line 7: the temporary pair, hoisted out of
// the loop; line 3: the running stats).
//   n      = RMS_{g_attn}(x)                                   (Sec. 2.2, first display)
//   q      = qkRMS_{g_q}(W_q n),  k~ = qkRMS_{g_k}(W_k n),  v~ = W_v n
//   (m,l,o) = state after UpdateTile(q_t, k~_t, v~_t) on (-inf, 0, 0): m = s<q,k~>, l = 1, o = v~
// Folding the temporary pair in here (Algorithm 1 does it as the first step of iteration t) is
// exact: the online-softmax merge does not depend on the order of the contributions.
// This file holds the SIMT projection used in fp32 mode and as the generic path; bf16 with d a
// multiple of 128 takes the tensor-core projection in rt_prepass_tc.cu.
#include "rt_kernels.h"

namespace rt {

// ---- n = RMS(x) (or a copy when pre-norm is off), position-major rows m = r*B + b ----------
template <typename T>
__global__ void rms_rows_kernel(const PrepassParams p) {
  grid_dep_sync();
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (m >= p.N * p.B) return;
  const int r = m / p.B, b = m % p.B;
  const T* xr = reinterpret_cast<const T*>(p.x) + (size_t)b * p.x_bs + (size_t)r * p.x_ts;
  T* out = reinterpret_cast<T*>(p.n) + (size_t)m * p.d;
  const T* g = reinterpret_cast<const T*>(p.g_attn);
  float ss = 0.f;
  for (int k = lane; k < p.d; k += 32) { const float v = to_f(xr[k]); ss += v * v; }
  ss = warp_sum(ss);
  const bool pre = (p.norm_flags & RT_NORM_PRE) != 0;
  const float rs = pre ? rsqrtf(ss / (float)p.d + p.eps) : 1.0f;
  for (int k = lane; k < p.d; k += 32) out[k] = from_f<T>(to_f(xr[k]) * rs * (pre ? gain_at(g, k) : 1.0f));
}

// ---- SIMT projection: C[m, col] = sum_k n[m,k] W[col,k], one head (64 columns) per CTA -----
constexpr int kGM = 64, kGN = 64, kGK = 16;

template <typename T>
__global__ void __launch_bounds__(256) qkv_gemm_simt_kernel(const PrepassParams p) {
  __shared__ float As[kGK][kGM + 4];
  __shared__ float Bs[kGK][kGN + 4];
  __shared__ float ssq[kGM][17];
  const int M = p.N * p.B, d = p.d;
  const int heads = d / kHeadDim;
  const int which = blockIdx.y / heads;        // 0: q, 1: k~, 2: v~
  if (p.mats && !((p.mats >> which) & 1)) return;
  const int head = blockIdx.y % heads;
  const int m0 = blockIdx.x * kGM;
  const T* W = reinterpret_cast<const T*>(which == 0 ? p.w_q : (which == 1 ? p.w_k : p.w_v)) + (size_t)head * kHeadDim * d;
  const T* A = reinterpret_cast<const T*>(p.n);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int lr = tid >> 2, lk = (tid & 3) * 4;    // each thread loads 4 consecutive k of one row
  for (int k0 = 0; k0 < d; k0 += kGK) {
    {
      const int m = m0 + lr;
      float f[4] = {0.f, 0.f, 0.f, 0.f};
      if (m < M) reinterpret_cast<const Vec4<T>*>(A + (size_t)m * d + k0 + lk)->to_float(f);
#pragma unroll
      for (int i = 0; i < 4; ++i) As[lk + i][lr] = f[i];
      float g[4];
      reinterpret_cast<const Vec4<T>*>(W + (size_t)lr * d + k0 + lk)->to_float(g);
#pragma unroll
      for (int i = 0; i < 4; ++i) Bs[lk + i][lr] = g[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kGK; ++kk) {
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
  // epilogue: per-row, per-head RMS for q and k~
  const bool qkn = (p.norm_flags & RT_NORM_QK) != 0 && which < 2;
  if (qkn) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) s += acc[i][j] * acc[i][j];
      ssq[ty * 4 + i][tx] = s;
    }
    __syncthreads();
  }
  const T* g = reinterpret_cast<const T*>(which == 0 ? p.g_q : p.g_k);
  T* out = reinterpret_cast<T*>(which == 0 ? p.q : (which == 1 ? p.kt : p.vt));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    float rs = 1.0f;
    if (qkn) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) s += ssq[ty * 4 + i][j];
      rs = rsqrtf(s * (1.0f / kHeadDim) + p.eps);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = head * kHeadDim + tx * 4 + j;
      out[(size_t)m * d + col] = from_f<T>(acc[i][j] * rs * (qkn ? gain_at(g, col) : 1.0f));
    }
  }
}

// ---- running stats seeded with the temporary pair ------------------------------------------
template <typename T>
__global__ void state_init_kernel(const PrepassParams p) {
  const int lane = threadIdx.x & 31;
  const long long u = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (m, h)
  const long long total = (long long)p.N * p.B * p.H;
  if (u >= total) return;
  const long long m = u / p.H;
  const int h = (int)(u % p.H);
  const size_t off = (size_t)m * p.d + h * kHeadDim + 2 * lane;
  const T* q = reinterpret_cast<const T*>(p.q) + off;
  const T* kt = reinterpret_cast<const T*>(p.kt) + off;
  const T* vt = reinterpret_cast<const T*>(p.vt) + off;
  const float dot = warp_sum(to_f(q[0]) * to_f(kt[0]) + to_f(q[1]) * to_f(kt[1]));
  *reinterpret_cast<float2*>(p.st_o + off) = make_float2(to_f(vt[0]), to_f(vt[1]));
  if (lane == 0) {
    p.st_m[u] = dot * p.scale_log2;
    p.st_l[u] = 1.0f;
  }
}

template <typename T>
static cudaError_t prepass_typed(const PrepassParams& p, cudaStream_t s) {
  const int M = p.N * p.B;
  if (!p.skip_rms) {
    const cudaError_t e = launch_chained(rms_rows_kernel<T>, dim3(ceil_div(M, 8)), dim3(256), 0, s, p.chained != 0, p);
    if (e != cudaSuccess) return e;
  }
  if (sizeof(T) == 2 && qkv_gemm_tc_supported(p)) {
    const cudaError_t e = qkv_gemm_tc_launch(p, p.sync, s);
    if (e != cudaSuccess) return e;
  } else {
    dim3 grid(ceil_div(M, kGM), 3 * (p.d / kHeadDim));
    qkv_gemm_simt_kernel<T><<<grid, 256, 0, s>>>(p);
  }
  if (!p.no_seed) {
    const long long units = (long long)M * p.H;
    state_init_kernel<T><<<(unsigned)((units + 7) / 8), 256, 0, s>>>(p);
  }
  return cudaGetLastError();
}

cudaError_t prepass_launch(int dtype, const PrepassParams& p, cudaStream_t s) {
  return dtype == RT_BF16 ? prepass_typed<__nv_bfloat16>(p, s) : prepass_typed<float>(p, s);
}

}  // namespace rt
