// Backward pass of one RT layer (Sec. 6, "The backward pass"; activation checkpointing as in Sec. 6).
//
// Given the layer input x, its outputs z (kept anyway: they are the next layer's input) and dL/dz, the call
//   1. rebuilds every intermediate in one parallel sweep (persistent pairs from z, queries and temporary pairs from x,
//      attention values and their log-sum-exp, the chain h, u, W_up u),
//   2. walks the positions in reverse and accumulates ONLY d(k_j, v_j): position i needs the final dL/dz_i, which
//      needs d(k_i, v_i) complete; pairs of other leaves get their share from the tiles of Algorithm 1 run backwards
//      (the same tiles, visited in reverse order, each as one launch over all its keys),
//   3. computes everything else -- dq, the temporary pairs, dx and all parameter gradients -- as large products over
//      all rows at once.
// The reverse loop and the attention terms are fp32 on CUDA cores; the products over all rows of stages 1 and 3 run on
// the tensor cores (bf16 copies of the operands, fp32 accumulation) when the storage type is bf16.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "rt_common.cuh"
#include "rt_kernels.h"

namespace rt {
namespace {

// ------------------------------------------------------------------------------------------------ generic product
// C[m, n] = alpha * sum_k A(m, k) Bm(k, n)  (+ C when accumulate), A(m,k) = A[m*a_rs + k*a_cs], Bm(k,n) = Bm[k*b_rs + n*b_cs].
template <typename TA, typename TB>
__global__ void __launch_bounds__(256) gemm_kernel(int M, int N, int K, const TA* __restrict__ A, long long a_rs, long long a_cs,
                                                   const TB* __restrict__ Bm, long long b_rs, long long b_cs,
                                                   float* __restrict__ C, long long ldc, float alpha, int accumulate) {
  __shared__ float As[16][68];
  __shared__ float Bs[16][68];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      int m, k;
      if (a_cs == 1) { k = t & 15; m = (t >> 4) + 16 * it; } else { m = t & 63; k = (t >> 6) + 4 * it; }
      float v = 0.f;
      if (m0 + m < M && k0 + k < K) v = to_f(A[(long long)(m0 + m) * a_rs + (long long)(k0 + k) * a_cs]);
      As[k][m] = v;
      int n;
      if (b_cs == 1) { n = t & 63; k = (t >> 6) + 4 * it; } else { k = t & 15; n = (t >> 4) + 16 * it; }
      v = 0.f;
      if (n0 + n < N && k0 + k < K) v = to_f(Bm[(long long)(k0 + k) * b_rs + (long long)(n0 + n) * b_cs]);
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < M && n < N) {
        float* c = C + (long long)m * ldc + n;
        *c = (accumulate ? *c : 0.f) + alpha * acc[i][j];
      }
    }
}

template <typename TA, typename TB>
cudaError_t gemm(int M, int N, int K, const TA* A, long long a_rs, long long a_cs, const TB* Bm, long long b_rs, long long b_cs,
                 float* C, long long ldc, float alpha, bool accumulate, cudaStream_t s) {
  gemm_kernel<TA, TB><<<dim3(ceil_div(N, 64), ceil_div(M, 64)), 256, 0, s>>>(M, N, K, A, a_rs, a_cs, Bm, b_rs, b_cs, C, ldc, alpha,
                                                                              accumulate ? 1 : 0);
  return cudaGetLastError();
}

// bf16 operands of the tensor-core products (bf16 storage only): a copy, or a transposed copy, of an fp32 / bf16 array
__global__ void to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, long long n) {
  grid_dep_sync();
  const long long idx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (idx + 3 < n) {
    const float4 v = *reinterpret_cast<const float4*>(in + idx);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(out + idx) = make_uint2(*reinterpret_cast<unsigned*>(&a), *reinterpret_cast<unsigned*>(&b));
  } else {
    for (long long j = idx; j < n; ++j) out[j] = __float2bfloat16_rn(in[j]);
  }
}
// out[c * R + r] = in[r * C + c]
template <typename TI>
__global__ void transpose_bf16_kernel(const TI* __restrict__ in, long long R, int C, __nv_bfloat16* __restrict__ out) {
  __shared__ float tile[32][33];
  const long long r0 = (long long)blockIdx.y * 32;
  const int c0 = blockIdx.x * 32;
  for (int j = threadIdx.y; j < 32; j += 8) {
    const long long r = r0 + j;
    const int c = c0 + threadIdx.x;
    tile[j][threadIdx.x] = (r < R && c < C) ? to_f(in[r * C + c]) : 0.f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    const int c = c0 + j;
    const long long r = r0 + threadIdx.x;
    if (r < R && c < C) out[(long long)c * R + r] = __float2bfloat16_rn(tile[threadIdx.x][j]);
  }
}

// ------------------------------------------------------------------------------------------------ RMS forward / backward
// Row r = i*B + b of a [B, N, *] array sits at b*bs + i*ts; position-major fp32 buffers use bs = width, ts = B*width.
__device__ __forceinline__ long long row_at(long long r, int B, long long bs, long long ts) { return (r % B) * bs + (r / B) * ts; }

// y = g u / sqrt(mean_G(u^2) + eps) over groups of G entries (G = d: RMS of Sec. 2; G = 64: qkRMS per head); copy when !enable.
template <typename TI, typename TG>
__global__ void norm_fwd_kernel(const TI* __restrict__ in, long long bs, long long ts, int B, const TG* __restrict__ g,
                                float* __restrict__ out, long long rows, int d, int G, float eps, int enable) {
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, groups = d / G;
  if (wid >= rows * groups) return;
  const long long r = wid / groups;
  const int c0 = (int)(wid % groups) * G;
  const TI* src = in + row_at(r, B, bs, ts) + c0;
  float* dst = out + r * d + c0;
  float ss = 0.f;
  for (int e = lane; e < G; e += 32) { const float v = to_f(src[e]); ss = fmaf(v, v, ss); }
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / G + eps);
  for (int e = lane; e < G; e += 32) dst[e] = enable ? to_f(src[e]) * inv * gain_at(g, c0 + e) : to_f(src[e]);
}

// With y = g u inv, inv = (mean(u^2)+eps)^(-1/2), t = g dy and uh = u inv:  du = inv (t - uh mean(t uh)),  dg += dy uh.
// out = (add ? add : 0) + du;  gprod (=|+=) dy uh.  out and gprod may each be NULL.  !enable: du = dy.
// out_bf (optional): a bf16 copy of bf_scale * out, [rows, d], the operand of the tensor-core product that follows.
template <typename TU, typename TG>
__global__ void norm_bwd_kernel(const float* dy, const TU* __restrict__ u, long long u_bs, long long u_ts, int B,
                                const TG* __restrict__ g, const float* add, float* out, long long o_bs, long long o_ts,
                                float* gprod, int gprod_acc, long long rows, int d, int G, float eps, int enable,
                                __nv_bfloat16* out_bf = nullptr, float bf_scale = 1.f) {
  grid_dep_sync();
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, groups = d / G;
  if (wid >= rows * groups) return;
  const long long r = wid / groups;
  const int c0 = (int)(wid % groups) * G;
  const float* dyr = dy + r * d + c0;
  const TU* ur = u + row_at(r, B, u_bs, u_ts) + c0;
  float ss = 0.f, tu = 0.f;
  if (enable) {
    for (int e = lane; e < G; e += 32) {
      const float v = to_f(ur[e]);
      ss = fmaf(v, v, ss);
      tu = fmaf(dyr[e] * gain_at(g, c0 + e), v, tu);
    }
    ss = warp_sum(ss); tu = warp_sum(tu);
  }
  const float inv = rsqrtf(ss / G + eps);
  const float mean = tu * inv / G;
  for (int e = lane; e < G; e += 32) {
    float du = dyr[e], gp = 0.f;
    if (enable) {
      const float uh = to_f(ur[e]) * inv;
      du = inv * (dyr[e] * gain_at(g, c0 + e) - uh * mean);
      gp = dyr[e] * uh;
    }
    const float res = (add ? add[r * d + c0 + e] : 0.f) + du;
    if (out) out[row_at(r, B, o_bs, o_ts) + c0 + e] = res;
    if (out_bf) out_bf[r * d + c0 + e] = __float2bfloat16_rn(res * bf_scale);   // operand copy for the next product
    if (gprod) gprod[r * d + c0 + e] = (gprod_acc ? gprod[r * d + c0 + e] : 0.f) + gp;
  }
}

// The same backward of a full-width RMS (G = d) with one CTA of 256 threads per row: for the few rows of one position
// of a wide batch, where a warp per row would leave the GPU idle.
template <typename TU, typename TG>
__global__ void __launch_bounds__(256) norm_bwd_row_kernel(const float* dy, const TU* __restrict__ u, long long u_bs, long long u_ts, int B,
                                                           const TG* __restrict__ g, const float* add, float* out, int d, float eps,
                                                           int enable, __nv_bfloat16* out_bf, float bf_scale) {
  grid_dep_sync();
  __shared__ float red[2][8];
  const long long r = blockIdx.x;
  const int tid = threadIdx.x;
  const float* dyr = dy + r * d;
  const TU* ur = u + row_at(r, B, u_bs, u_ts);
  float ss = 0.f, tu = 0.f;
  if (enable) {
    for (int e = tid; e < d; e += 256) {
      const float v = to_f(ur[e]);
      ss = fmaf(v, v, ss);
      tu = fmaf(dyr[e] * gain_at(g, e), v, tu);
    }
    ss = warp_sum(ss); tu = warp_sum(tu);
    if ((tid & 31) == 0) { red[0][tid >> 5] = ss; red[1][tid >> 5] = tu; }
    __syncthreads();
    ss = 0.f; tu = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { ss += red[0][w]; tu += red[1][w]; }
  }
  const float inv = rsqrtf(ss / d + eps), mean = tu * inv / d;
  for (int e = tid; e < d; e += 256) {
    float du = dyr[e];
    if (enable) du = inv * (dyr[e] * gain_at(g, e) - to_f(ur[e]) * inv * mean);
    const float res = add[r * d + e] + du;
    out[r * d + e] = res;
    if (out_bf) out_bf[r * d + e] = __float2bfloat16_rn(res * bf_scale);
  }
}

// column sums of a [rows, d] array in two fixed-order steps
__global__ void col_partial_kernel(const float* __restrict__ a, long long rows, int d, float* __restrict__ part, int P) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  const long long chunk = (rows + P - 1) / P, r0 = blockIdx.y * chunk, r1 = r0 + chunk < rows ? r0 + chunk : rows;
  float s = 0.f;
  for (long long r = r0; r < r1; ++r) s += a[r * d + c];
  part[(long long)blockIdx.y * d + c] = s;
}
__global__ void col_final_kernel(const float* __restrict__ part, int P, int d, float* out, int accumulate) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  float s = 0.f;
  for (int p = 0; p < P; ++p) s += part[(long long)p * d + c];
  out[c] = (accumulate ? out[c] : 0.f) + s;
}

// h = x + alpha a  (x [B,N,d] storage type, a and h position-major fp32)
template <typename T>
__global__ void residual_kernel(const T* __restrict__ x, long long bs, long long ts, int B, const float* __restrict__ a, float alpha,
                                float* __restrict__ h, long long rows, int d) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * d) return;
  const long long r = idx / d;
  const int c = (int)(idx % d);
  h[idx] = to_f(x[row_at(r, B, bs, ts) + c]) + alpha * a[idx];
}

__device__ __forceinline__ float gelu_f(float a) { return 0.5f * a * (1.f + erff(a * 0.70710678118654752f)); }
// d/da [a Phi(a)] = Phi(a) + a phi(a)
__device__ __forceinline__ float gelu_grad_f(float a) {
  return 0.5f * (1.f + erff(a * 0.70710678118654752f)) + a * 0.3989422804014327f * __expf(-0.5f * a * a);
}
// four consecutive entries per thread (n a multiple of 4: d_ff is)
__global__ void gelu_bwd_kernel(float* __restrict__ dg, const float* __restrict__ a, long long n, __nv_bfloat16* out_bf) {
  grid_dep_sync();
  const long long idx = 4 * ((long long)blockIdx.x * blockDim.x + threadIdx.x);
  if (idx < n) {
    const float4 g = *reinterpret_cast<const float4*>(dg + idx), x = *reinterpret_cast<const float4*>(a + idx);
    const float4 v = make_float4(g.x * gelu_grad_f(x.x), g.y * gelu_grad_f(x.y), g.z * gelu_grad_f(x.z), g.w * gelu_grad_f(x.w));
    *reinterpret_cast<float4*>(dg + idx) = v;
    if (out_bf) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      *reinterpret_cast<uint2*>(out_bf + idx) = make_uint2(*reinterpret_cast<const unsigned*>(&lo), *reinterpret_cast<const unsigned*>(&hi));
    }
  }
}
__global__ void gelu_kernel(const float* __restrict__ a, float* __restrict__ out, long long n) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < n) out[idx] = gelu_f(a[idx]);
}

// ------------------------------------------------------------------------------------------------ attention
struct AttnBufs {
  const float *q, *k, *v, *kt, *vt;        // position-major [rows, d]
  float *lse, *D;                          // [rows, H]: log2-sum-exp of the logits (log2 units), <dc, c> per head
  float *c;                                // [rows, d] attention value
  const float* dc;                         // [rows, d] gradient of the attention value
  float *dK, *dV, *dkt, *dvt, *dq;
  const float* alibi;                      // [H] or NULL
  float scale, scale_log2;
  int B, H, d, N;
};

// ---- eight lanes per (query, key) pair -------------------------------------------------------------------------------
// The three all-pairs kernels below split a warp into four groups of eight lanes; a group works on one pair at a time,
// each lane holding eight consecutive entries of the 64-wide head, so a dot product costs three shuffles for four pairs.
struct F8 { float v[8]; };
__device__ __forceinline__ F8 ld8(const float* p) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  return F8{{a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w}};
}
__device__ __forceinline__ void st8(float* p, const F8& x) {
  *reinterpret_cast<float4*>(p) = make_float4(x.v[0], x.v[1], x.v[2], x.v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(x.v[4], x.v[5], x.v[6], x.v[7]);
}
__device__ __forceinline__ float dot8(const F8& a, const F8& b) {
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) s = fmaf(a.v[e], b.v[e], s);
  return s;
}
__device__ __forceinline__ float group_sum(float v) {          // over the eight lanes of a group
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  return v;
}
__device__ __forceinline__ float across_groups_sum(float v) {   // over the four groups, lane by lane
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  v += __shfl_xor_sync(0xffffffffu, v, 16);
  return v;
}

// The softmax of Sec. 2.2 for every (position, sequence, head): attention value c and log2-sum-exp of the logits over
// the pairs j < i and the temporary pair.  One warp per FOUR consecutive positions of one (sequence, head): group g is
// position 4 iq + g, all four groups read the same pair j in the same instruction (one fetch, broadcast), and the warps
// of a CTA are consecutive position quads of the same (sequence, head), so the pair rows stay in L1.
__global__ void attn_stats_kernel(AttnBufs a) {
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, g = lane >> 3, t = lane & 7;
  const int NQ = (a.N + 3) / 4;
  if (wid >= (long long)NQ * a.B * a.H) return;
  const int iq = (int)(wid % NQ), h = (int)((wid / NQ) % a.H), b = (int)(wid / ((long long)NQ * a.H));
  const int i = 4 * iq + g;
  const bool live = i < a.N;
  const long long col = (long long)h * kHeadDim + 8 * t;
  const long long ri = ((long long)(live ? i : a.N - 1) * a.B + b) * a.d + col;
  const long long rstride = (long long)a.B * a.d;
  const F8 q = ld8(a.q + ri);
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  float m = -INFINITY, l = 0.f;
  F8 o = {};
  const int jend = 4 * iq + 3 < a.N - 1 ? 4 * iq + 3 : a.N - 1;   // pairs needed by the last position of the quad
  long long rj = (long long)b * a.d + col;
  auto update = [&](int j, float sd, const F8& vv) {
    if (j < i) {
      const float sc = sd * a.scale_log2 - slope * (float)(i - j);
      const float mn = fmaxf(m, sc);
      const float corr = exp2f(m - mn), p = exp2f(sc - mn);
      l = l * corr + p;
#pragma unroll
      for (int e = 0; e < 8; ++e) o.v[e] = fmaf(p, vv.v[e], o.v[e] * corr);
      m = mn;
    }
  };
  int j = 0;
  for (; j + 4 <= jend; j += 4, rj += 4 * rstride) {          // four pairs in flight
    F8 vv[4];
    float sd[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const F8 kk = ld8(a.k + rj + u * rstride);
      vv[u] = ld8(a.v + rj + u * rstride);
      sd[u] = dot8(q, kk);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) sd[u] = group_sum(sd[u]);
#pragma unroll
    for (int u = 0; u < 4; ++u) update(j + u, sd[u], vv[u]);
  }
  for (; j < jend; ++j, rj += rstride) {
    const F8 kk = ld8(a.k + rj), vv = ld8(a.v + rj);
    update(j, group_sum(dot8(q, kk)), vv);
  }
  const F8 kt = ld8(a.kt + ri), vt = ld8(a.vt + ri);           // the temporary pair of the position itself
  const float st = group_sum(dot8(q, kt)) * a.scale_log2;
  const float mf = fmaxf(m, st);
  const float w = m == -INFINITY ? 0.f : exp2f(m - mf), pt = exp2f(st - mf);
  l = l * w + pt;
  const float inv = 1.f / l;
  F8 c;
#pragma unroll
  for (int e = 0; e < 8; ++e) c.v[e] = (o.v[e] * w + pt * vt.v[e]) * inv;
  if (live) {
    st8(a.c + ri, c);
    if (t == 0) a.lse[((long long)i * a.B + b) * a.H + h] = mf + log2f(l);
  }
}

// Tensor-core route of the attention statistics (bf16 storage): the running softmax state (o, m in log2 units, l) is
// seeded with the temporary pair here, advanced over all earlier pairs by the forward pass's own tile kernels
// (Algorithm 2), and turned into c = o / l and the log2-sum-exp afterwards.  One warp per (position, sequence, head).
__global__ void stats_seed_kernel(AttnBufs a, float* st_o, float* st_m, float* st_l) {
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (long long)a.N * a.B * a.H) return;
  const int h = (int)(wid % a.H);
  const long long row = wid / a.H;
  const long long at = row * a.d + (long long)h * kHeadDim + 2 * lane;
  const float2 q = *reinterpret_cast<const float2*>(a.q + at), kt = *reinterpret_cast<const float2*>(a.kt + at);
  const float s = warp_sum(q.x * kt.x + q.y * kt.y) * a.scale_log2;
  *reinterpret_cast<float2*>(st_o + at) = *reinterpret_cast<const float2*>(a.vt + at);
  if (lane == 0) { st_m[row * a.H + h] = s; st_l[row * a.H + h] = 1.f; }
}
__global__ void stats_finish_kernel(AttnBufs a, float* st_o, float* st_m, const float* st_l) {
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (long long)a.N * a.B * a.H) return;
  const int h = (int)(wid % a.H);
  const long long row = wid / a.H;
  const long long at = row * a.d + (long long)h * kHeadDim + 2 * lane;
  const float l = st_l[row * a.H + h], inv = 1.f / l;
  float2 o = *reinterpret_cast<const float2*>(st_o + at);
  o.x *= inv; o.y *= inv;
  *reinterpret_cast<float2*>(st_o + at) = o;                   // c in place
  if (lane == 0) st_m[row * a.H + h] += log2f(l);              // log2-sum-exp in place
}

// State of the reverse loop written earlier in the SAME (cooperative) kernel by other CTAs must not come from L1.
template <bool COOP> __device__ __forceinline__ float ld_state(const float* p) { return COOP ? __ldcg(p) : *p; }
template <bool COOP> __device__ __forceinline__ float2 ld_state2(const float* p) {
  return COOP ? __ldcg(reinterpret_cast<const float2*>(p)) : *reinterpret_cast<const float2*>(p);
}

// In-leaf step of position i for one (key j in [s0, i], sequence, head), one warp: see attn_bwd_kv_kernel (self = 1).
template <bool COOP>
__device__ __forceinline__ void attn_self_task(const AttnBufs& a, int i, int j, int b, int h, int lane) {
  const long long col = (long long)h * kHeadDim + 2 * lane;
  const long long rj = ((long long)j * a.B + b) * a.d + col;
  const long long ri = ((long long)i * a.B + b) * a.d + col;
  const long long si = ((long long)i * a.B + b) * a.H + h;
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  const float2 dc = ld_state2<COOP>(a.dc + ri);
  const float2 cc = *reinterpret_cast<const float2*>(a.c + ri);
  const float2 q = *reinterpret_cast<const float2*>(a.q + ri);
  const float D = warp_sum(dc.x * cc.x + dc.y * cc.y);
  const float lse = a.lse[si];
  if (j == i) {
    if (lane == 0) a.D[si] = D;
    const float2 kk = *reinterpret_cast<const float2*>(a.kt + ri);
    const float2 vv = *reinterpret_cast<const float2*>(a.vt + ri);
    const float p = exp2f(warp_sum(q.x * kk.x + q.y * kk.y) * a.scale_log2 - lse);
    const float ds = p * (warp_sum(dc.x * vv.x + dc.y * vv.y) - D) * a.scale;
    *reinterpret_cast<float2*>(a.dkt + ri) = make_float2(ds * q.x, ds * q.y);
    *reinterpret_cast<float2*>(a.dvt + ri) = make_float2(p * dc.x, p * dc.y);
  } else {
    const float2 kk = *reinterpret_cast<const float2*>(a.k + rj);
    const float2 vv = *reinterpret_cast<const float2*>(a.v + rj);
    const float p = exp2f(warp_sum(q.x * kk.x + q.y * kk.y) * a.scale_log2 - slope * (float)(i - j) - lse);
    const float ds = p * (warp_sum(dc.x * vv.x + dc.y * vv.y) - D) * a.scale;
    float2 t = ld_state2<COOP>(a.dK + rj); t.x += ds * q.x; t.y += ds * q.y; *reinterpret_cast<float2*>(a.dK + rj) = t;
    t = ld_state2<COOP>(a.dV + rj); t.x += p * dc.x; t.y += p * dc.y; *reinterpret_cast<float2*>(a.dV + rj) = t;
  }
}

// In-leaf step of position i as a launch of its own (the one-launch-per-step form of the reverse loop): one warp per
// (key j in [k0, i], sequence, head), see attn_self_task.
__global__ void attn_bwd_kv_kernel(AttnBufs a, int i, int k0) {
  grid_dep_sync();
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (long long)(i + 1 - k0) * a.B * a.H) return;
  const int h = (int)(wid % a.H), b = (int)((wid / a.H) % a.B), j = k0 + (int)(wid / ((long long)a.H * a.B));
  attn_self_task<false>(a, i, j, b, h, lane);
}

// In-leaf step of position i for wide batches: one warp per (sequence, head) walks the pairs [k0, i) of the leaf, four at
// a time (a group of eight lanes per pair, which it owns: plain read-modify-write), then the temporary pair and D_i.
__global__ void attn_self_wide_kernel(AttnBufs a, int i, int k0) {
  grid_dep_sync();
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, g = lane >> 3, t = lane & 7;
  if (wid >= (long long)a.B * a.H) return;
  const int h = (int)(wid % a.H), b = (int)(wid / a.H);
  const long long col = (long long)h * kHeadDim + 8 * t;
  const long long rstride = (long long)a.B * a.d;
  const long long ri = (long long)i * rstride + (long long)b * a.d + col;
  const long long si = ((long long)i * a.B + b) * a.H + h;
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  const F8 q = ld8(a.q + ri), dc = ld8(a.dc + ri), cc = ld8(a.c + ri);
  const float D = group_sum(dot8(dc, cc)), lse = a.lse[si];
  for (int j0 = k0; j0 < i; j0 += 4) {
    const int j = j0 + g;
    const bool valid = j < i;
    const long long rj = (long long)(valid ? j : k0) * rstride + (long long)b * a.d + col;
    const F8 kk = ld8(a.k + rj), vv = ld8(a.v + rj);
    F8 gk = ld8(a.dK + rj), gv = ld8(a.dV + rj);
    const float sd = group_sum(dot8(q, kk)), dp = group_sum(dot8(dc, vv));
    if (valid) {
      const float p = exp2f(sd * a.scale_log2 - slope * (float)(i - j) - lse);
      const float ds = p * (dp - D) * a.scale;
#pragma unroll
      for (int e = 0; e < 8; ++e) { gk.v[e] = fmaf(ds, q.v[e], gk.v[e]); gv.v[e] = fmaf(p, dc.v[e], gv.v[e]); }
      st8(a.dK + rj, gk); st8(a.dV + rj, gv);
    }
  }
  const F8 kt = ld8(a.kt + ri), vt = ld8(a.vt + ri);
  const float p = exp2f(group_sum(dot8(q, kt)) * a.scale_log2 - lse);
  const float ds = p * (group_sum(dot8(dc, vt)) - D) * a.scale;
  if (g == 0) {
    F8 o1, o2;
#pragma unroll
    for (int e = 0; e < 8; ++e) { o1.v[e] = ds * q.v[e]; o2.v[e] = p * dc.v[e]; }
    st8(a.dkt + ri, o1); st8(a.dvt + ri, o2);
    if (t == 0) a.D[si] = D;
  }
}

// A tile of Algorithm 1 backwards: the pairs [k0, k1) receive the share of the queries [q0, q1) (all later positions):
//   p = exp2(logit - lse_i), ds = p (<dc_i, v_j> - D_i), dk_j += scale ds q_i, dv_j += p dc_i.
// One warp per (key j, sequence, head) holds k_j, v_j; its four groups take the queries q0 + g, q0 + g + 4, ... and the
// four partial sums are added in a fixed order at the end (no atomics).
__global__ void attn_bwd_kv_tile_kernel(AttnBufs a, int q0, int q1, int k0, int k1) {
  grid_dep_sync();
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int P = k1 - k0;
  if (wid >= (long long)P * a.B * a.H) return;
  // consecutive warps = consecutive keys of one (sequence, head): the warps of a CTA walk the same query rows together
  const int j = k0 + (int)(wid % P), h = (int)((wid / P) % a.H), b = (int)(wid / ((long long)P * a.H));
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  // a tile of Algorithm 1 backwards: group g takes the queries q0 + g, q0 + g + 4, ...
  const int g = lane >> 3, t = lane & 7;
  const long long col8 = (long long)h * kHeadDim + 8 * t;
  const long long rj8 = ((long long)j * a.B + b) * a.d + col8;
  const long long rstride = (long long)a.B * a.d, sstride = (long long)a.B * a.H;
  const F8 kk = ld8(a.k + rj8), vv = ld8(a.v + rj8);
  F8 dk = {}, dv = {};
  for (int i0 = q0; i0 < q1; i0 += 4) {
    const int i = i0 + g;
    const bool valid = i < q1;
    const int ic = valid ? i : q0;
    const long long ri = (long long)ic * rstride + (long long)b * a.d + col8;
    const long long si = (long long)ic * sstride + (long long)b * a.H + h;
    const F8 q = ld8(a.q + ri), dc = ld8(a.dc + ri);
    const float lse = a.lse[si], D = a.D[si];
    const float sd = group_sum(dot8(q, kk)), dp = group_sum(dot8(dc, vv));
    if (valid) {
      const float p = exp2f(sd * a.scale_log2 - slope * (float)(i - j) - lse);
      const float ds = p * (dp - D) * a.scale;
#pragma unroll
      for (int e = 0; e < 8; ++e) { dk.v[e] = fmaf(ds, q.v[e], dk.v[e]); dv.v[e] = fmaf(p, dc.v[e], dv.v[e]); }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) { dk.v[e] = across_groups_sum(dk.v[e]); dv.v[e] = across_groups_sum(dv.v[e]); }
  if (g == 0) {
    F8 cur = ld8(a.dK + rj8);
#pragma unroll
    for (int e = 0; e < 8; ++e) cur.v[e] += dk.v[e];
    st8(a.dK + rj8, cur);
    cur = ld8(a.dV + rj8);
#pragma unroll
    for (int e = 0; e < 8; ++e) cur.v[e] += dv.v[e];
    st8(a.dV + rj8, cur);
  }
}

// The same tile with 64 x 64 blocks of (query, key) pairs held in shared memory (key counts that are multiples of 64):
// one CTA per (64 keys, sequence, head); for each block of 64 queries it forms S = Q K^T and dP = dC V^T as 4 x 4
// register tiles per thread, P and dS from them, and adds dS^T Q to dk and P^T dC to dv -- every operand row is fetched
// once per block instead of once per pair.  Queries in order, fixed summation order, no atomics.
constexpr int kPB = 64, kPBS = kPB + 1;                        // block edge, padded row stride in shared memory
constexpr size_t kPairBlockSmem = (6 * kPB * kPBS + 2 * kPB) * sizeof(float);
__global__ void __launch_bounds__(256) attn_bwd_kv_block_kernel(AttnBufs a, int q0, int q1, int k0, int k1) {
  grid_dep_sync();
  extern __shared__ __align__(16) float sm[];
  float *Qs = sm, *Cs = Qs + kPB * kPBS, *Ks = Cs + kPB * kPBS, *Vs = Ks + kPB * kPBS, *Ps = Vs + kPB * kPBS, *Ss = Ps + kPB * kPBS;
  float *lse_s = Ss + kPB * kPBS, *D_s = lse_s + kPB;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int b = blockIdx.y / a.H, h = blockIdx.y % a.H;
  const int kb = k0 + kPB * blockIdx.x;
  const long long col0 = (long long)b * a.d + (long long)h * kHeadDim;
  const long long rstride = (long long)a.B * a.d;
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  for (int idx = tid; idx < kPB * 16; idx += 256) {             // the 64 keys of this CTA: rows of 64 entries as 16 float4
    const int j = idx >> 4, e4 = (idx & 15) * 4;
    const float4 kk = *reinterpret_cast<const float4*>(a.k + (long long)(kb + j) * rstride + col0 + e4);
    const float4 vv = *reinterpret_cast<const float4*>(a.v + (long long)(kb + j) * rstride + col0 + e4);
    float* kd = Ks + j * kPBS + e4; kd[0] = kk.x; kd[1] = kk.y; kd[2] = kk.z; kd[3] = kk.w;
    float* vd = Vs + j * kPBS + e4; vd[0] = vv.x; vd[1] = vv.y; vd[2] = vv.z; vd[3] = vv.w;
  }
  float dk[4][4] = {}, dv[4][4] = {};                           // keys ty + 16 jj, entries tx + 16 ee
  for (int qb = q0; qb < q1; qb += kPB) {
    const int nq = q1 - qb < kPB ? q1 - qb : kPB;
    __syncthreads();                                            // the previous block's tiles are no longer read
    for (int idx = tid; idx < kPB * 16; idx += 256) {
      const int i = idx >> 4, e4 = (idx & 15) * 4;
      float4 qq = make_float4(0.f, 0.f, 0.f, 0.f), cc = qq;
      if (i < nq) {
        qq = *reinterpret_cast<const float4*>(a.q + (long long)(qb + i) * rstride + col0 + e4);
        cc = *reinterpret_cast<const float4*>(a.dc + (long long)(qb + i) * rstride + col0 + e4);
      }
      float* qd = Qs + i * kPBS + e4; qd[0] = qq.x; qd[1] = qq.y; qd[2] = qq.z; qd[3] = qq.w;
      float* cd = Cs + i * kPBS + e4; cd[0] = cc.x; cd[1] = cc.y; cd[2] = cc.z; cd[3] = cc.w;
    }
    if (tid < kPB) {
      const long long si = ((long long)(qb + (tid < nq ? tid : 0)) * a.B + b) * a.H + h;
      lse_s[tid] = a.lse[si]; D_s[tid] = a.D[si];
    }
    __syncthreads();
    // S and dP: queries ty + 16 ii, keys tx + 16 jj
    float sv[4][4] = {}, dp[4][4] = {};
#pragma unroll 4
    for (int e = 0; e < kPB; ++e) {
      float qv[4], cv[4], kv[4], vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        qv[u] = Qs[(ty + 16 * u) * kPBS + e]; cv[u] = Cs[(ty + 16 * u) * kPBS + e];
        kv[u] = Ks[(tx + 16 * u) * kPBS + e]; vv[u] = Vs[(tx + 16 * u) * kPBS + e];
      }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) { sv[ii][jj] = fmaf(qv[ii], kv[jj], sv[ii][jj]); dp[ii][jj] = fmaf(cv[ii], vv[jj], dp[ii][jj]); }
    }
#pragma unroll
    for (int ii = 0; ii < 4; ++ii)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int il = ty + 16 * ii, jl = tx + 16 * jj;
        float p = 0.f, ds = 0.f;
        if (il < nq) {
          p = exp2f(sv[ii][jj] * a.scale_log2 - slope * (float)(qb + il - kb - jl) - lse_s[il]);
          ds = p * (dp[ii][jj] - D_s[il]) * a.scale;
        }
        Ps[il * kPBS + jl] = p; Ss[il * kPBS + jl] = ds;
      }
    __syncthreads();
    // dk += dS^T Q, dv += P^T dC: keys ty + 16 jj, entries tx + 16 ee
#pragma unroll 4
    for (int i = 0; i < kPB; ++i) {
      float sj[4], pj[4], qe[4], ce[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        sj[u] = Ss[i * kPBS + ty + 16 * u]; pj[u] = Ps[i * kPBS + ty + 16 * u];
        qe[u] = Qs[i * kPBS + tx + 16 * u]; ce[u] = Cs[i * kPBS + tx + 16 * u];
      }
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
#pragma unroll
        for (int ee = 0; ee < 4; ++ee) { dk[jj][ee] = fmaf(sj[jj], qe[ee], dk[jj][ee]); dv[jj][ee] = fmaf(pj[jj], ce[ee], dv[jj][ee]); }
    }
  }
#pragma unroll
  for (int jj = 0; jj < 4; ++jj)
#pragma unroll
    for (int ee = 0; ee < 4; ++ee) {
      const long long at = (long long)(kb + ty + 16 * jj) * rstride + col0 + tx + 16 * ee;
      a.dK[at] += dk[jj][ee];
      a.dV[at] += dv[jj][ee];
    }
}

// Gradient of the queries, all positions at once: dq_i = scale (sum_{j<i} ds_ij k_j + ds_ii~ k~_i).  Same layout as
// attn_stats_kernel: one warp per four consecutive positions of one (sequence, head), group g = position 4 iq + g.
__global__ void attn_bwd_q_kernel(AttnBufs a) {
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, g = lane >> 3, t = lane & 7;
  const int NQ = (a.N + 3) / 4;
  if (wid >= (long long)NQ * a.B * a.H) return;
  const int iq = (int)(wid % NQ), h = (int)((wid / NQ) % a.H), b = (int)(wid / ((long long)NQ * a.H));
  const int i = 4 * iq + g;
  const bool live = i < a.N;
  const int ic = live ? i : a.N - 1;
  const long long col = (long long)h * kHeadDim + 8 * t;
  const long long ri = ((long long)ic * a.B + b) * a.d + col;
  const long long si = ((long long)ic * a.B + b) * a.H + h;
  const long long rstride = (long long)a.B * a.d;
  const F8 q = ld8(a.q + ri), dc = ld8(a.dc + ri);
  const float lse = a.lse[si], D = a.D[si];
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  F8 acc = {};
  const int jend = 4 * iq + 3 < a.N - 1 ? 4 * iq + 3 : a.N - 1;
  long long rj = (long long)b * a.d + col;
  int j = 0;
  for (; j + 4 <= jend; j += 4, rj += 4 * rstride) {          // four pairs in flight
    F8 kk[4];
    float sd[4], dp[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      kk[u] = ld8(a.k + rj + u * rstride);
      const F8 vv = ld8(a.v + rj + u * rstride);
      sd[u] = dot8(q, kk[u]); dp[u] = dot8(dc, vv);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) { sd[u] = group_sum(sd[u]); dp[u] = group_sum(dp[u]); }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (j + u < i) {
        const float ds = exp2f(sd[u] * a.scale_log2 - slope * (float)(i - j - u) - lse) * (dp[u] - D);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc.v[e] = fmaf(ds, kk[u].v[e], acc.v[e]);
      }
  }
  for (; j < jend; ++j, rj += rstride) {
    const F8 kk = ld8(a.k + rj), vv = ld8(a.v + rj);
    const float sd = group_sum(dot8(q, kk)), dp = group_sum(dot8(dc, vv));
    if (j < i) {
      const float ds = exp2f(sd * a.scale_log2 - slope * (float)(i - j) - lse) * (dp - D);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc.v[e] = fmaf(ds, kk.v[e], acc.v[e]);
    }
  }
  const F8 kt = ld8(a.kt + ri), vt = ld8(a.vt + ri);
  const float st = group_sum(dot8(q, kt)), dpt = group_sum(dot8(dc, vt));
  const float dst = exp2f(st * a.scale_log2 - lse) * (dpt - D);
  F8 out;
#pragma unroll
  for (int e = 0; e < 8; ++e) out.v[e] = (acc.v[e] + dst * kt.v[e]) * a.scale;
  if (live) st8(a.dq + ri, out);
}

// dq of all positions with 64 x 64 blocks of pairs in shared memory: one CTA per (64 queries, sequence, head) walks the
// key blocks up to its own (pairs j < i only), forms S and dP as register tiles, dS from them, and adds dS K to dq;
// the temporary pair of each position is added at the end.
constexpr size_t kPairBlockSmemQ = (5 * kPB * kPBS + 2 * kPB) * sizeof(float);
__global__ void __launch_bounds__(256) attn_bwd_q_block_kernel(AttnBufs a) {
  extern __shared__ __align__(16) float sm[];
  float *Qs = sm, *Cs = Qs + kPB * kPBS, *Ks = Cs + kPB * kPBS, *Vs = Ks + kPB * kPBS, *Ss = Vs + kPB * kPBS;
  float *lse_s = Ss + kPB * kPBS, *D_s = lse_s + kPB;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int b = blockIdx.y / a.H, h = blockIdx.y % a.H;
  const int qb = kPB * blockIdx.x;
  const int nq = a.N - qb < kPB ? a.N - qb : kPB;
  const long long col0 = (long long)b * a.d + (long long)h * kHeadDim;
  const long long rstride = (long long)a.B * a.d;
  const float slope = a.alibi ? a.alibi[h] * kLog2e : 0.f;
  for (int idx = tid; idx < kPB * 16; idx += 256) {
    const int i = idx >> 4, e4 = (idx & 15) * 4;
    float4 qq = make_float4(0.f, 0.f, 0.f, 0.f), cc = qq;
    if (i < nq) {
      qq = *reinterpret_cast<const float4*>(a.q + (long long)(qb + i) * rstride + col0 + e4);
      cc = *reinterpret_cast<const float4*>(a.dc + (long long)(qb + i) * rstride + col0 + e4);
    }
    float* qd = Qs + i * kPBS + e4; qd[0] = qq.x; qd[1] = qq.y; qd[2] = qq.z; qd[3] = qq.w;
    float* cd = Cs + i * kPBS + e4; cd[0] = cc.x; cd[1] = cc.y; cd[2] = cc.z; cd[3] = cc.w;
  }
  if (tid < kPB) {
    const long long si = ((long long)(qb + (tid < nq ? tid : 0)) * a.B + b) * a.H + h;
    lse_s[tid] = a.lse[si]; D_s[tid] = a.D[si];
  }
  float dq[4][4] = {};                                          // queries ty + 16 ii, entries tx + 16 ee
  const int k_end = qb + nq - 1;                                // pairs j < i <= qb + nq - 1
  for (int kb = 0; kb < k_end; kb += kPB) {
    const int nk = k_end - kb < kPB ? k_end - kb : kPB;
    __syncthreads();
    for (int idx = tid; idx < kPB * 16; idx += 256) {
      const int j = idx >> 4, e4 = (idx & 15) * 4;
      float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
      if (j < nk) {
        kk = *reinterpret_cast<const float4*>(a.k + (long long)(kb + j) * rstride + col0 + e4);
        vv = *reinterpret_cast<const float4*>(a.v + (long long)(kb + j) * rstride + col0 + e4);
      }
      float* kd = Ks + j * kPBS + e4; kd[0] = kk.x; kd[1] = kk.y; kd[2] = kk.z; kd[3] = kk.w;
      float* vd = Vs + j * kPBS + e4; vd[0] = vv.x; vd[1] = vv.y; vd[2] = vv.z; vd[3] = vv.w;
    }
    __syncthreads();
    float sv[4][4] = {}, dp[4][4] = {};
#pragma unroll 4
    for (int e = 0; e < kPB; ++e) {
      float qv[4], cv[4], kv[4], vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        qv[u] = Qs[(ty + 16 * u) * kPBS + e]; cv[u] = Cs[(ty + 16 * u) * kPBS + e];
        kv[u] = Ks[(tx + 16 * u) * kPBS + e]; vv[u] = Vs[(tx + 16 * u) * kPBS + e];
      }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) { sv[ii][jj] = fmaf(qv[ii], kv[jj], sv[ii][jj]); dp[ii][jj] = fmaf(cv[ii], vv[jj], dp[ii][jj]); }
    }
#pragma unroll
    for (int ii = 0; ii < 4; ++ii)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int il = ty + 16 * ii, jl = tx + 16 * jj;
        const int i = qb + il, j = kb + jl;
        float ds = 0.f;
        if (il < nq && j < i)
          ds = exp2f(sv[ii][jj] * a.scale_log2 - slope * (float)(i - j) - lse_s[il]) * (dp[ii][jj] - D_s[il]);
        Ss[il * kPBS + jl] = ds;
      }
    __syncthreads();
#pragma unroll 4
    for (int j = 0; j < kPB; ++j) {
      float si[4], ke[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { si[u] = Ss[(ty + 16 * u) * kPBS + j]; ke[u] = Ks[j * kPBS + tx + 16 * u]; }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int ee = 0; ee < 4; ++ee) dq[ii][ee] = fmaf(si[ii], ke[ee], dq[ii][ee]);
    }
  }
  // the temporary pair of each position: one warp per eight queries, then the scaled sum goes out
  __syncthreads();
  {
    const int warp = tid >> 5, lane = tid & 31;
    for (int il = warp; il < kPB; il += 8) {
      float ds = 0.f;
      if (il < nq) {
        const long long at = (long long)(qb + il) * rstride + col0;
        const float kt0 = a.kt[at + lane], kt1 = a.kt[at + lane + 32], vt0 = a.vt[at + lane], vt1 = a.vt[at + lane + 32];
        const float st = warp_sum(Qs[il * kPBS + lane] * kt0 + Qs[il * kPBS + lane + 32] * kt1);
        const float dpt = warp_sum(Cs[il * kPBS + lane] * vt0 + Cs[il * kPBS + lane + 32] * vt1);
        ds = exp2f(st * a.scale_log2 - lse_s[il]) * (dpt - D_s[il]);
      }
      if (lane == 0) Ss[il * kPBS] = ds;                        // column 0 of Ss: ds of the temporary pair
    }
  }
  __syncthreads();
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    const int il = ty + 16 * ii;
    if (il < nq) {
      const long long at = (long long)(qb + il) * rstride + col0;
#pragma unroll
      for (int ee = 0; ee < 4; ++ee) {
        const int e = tx + 16 * ee;
        a.dq[at + e] = (dq[ii][ee] + Ss[il * kPBS] * a.kt[at + e]) * a.scale;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------ the reverse loop's products
// One position i, the B rows of the batch: out[b, n] = alpha * (sum_k in1[b,k] W1[k,n] + sum_k in2[b,k] W2[k,n]) where the
// rows in1 (in2) are built by a prologue from the state of the reverse loop (mode), W = a weight matrix as stored
// ([its outputs, its inputs] = [K, Ncols]: the transposed product of the forward pass, read row by row).
enum { RM_PAIR = 1, RM_DOWN = 2, RM_UP = 3, RM_OUT = 4 };
constexpr int kRmThreads = 512, kRmWarps = kRmThreads / 32;   // rows (sequences) per task: RB = 4 or 8, a template parameter
struct RowmatParams {
  int mode, B, d, dff, i, K, Ncols;
  int cols;                               // columns per task: 16 or 32
  int nsplit;                             // RM_PAIR: 2 (task 0 = W_k with dk, task 1 = W_v with dv); RM_UP: parts of the contraction
  int norm_on, qk_on;                     // whether the prologue's RMS / qkRMS is active
  int n_in;                               // partial sums the prologue adds up (RM_DOWN: 2, RM_OUT: RM_UP's nsplit)
  float eps, alpha;
  const void *W1, *W2, *gain;             // storage type
  const void* z; long long z_bs, z_ts;    // layer output [B,N,d], storage type (RM_DOWN)
  const float* dz; long long dz_bs, dz_ts;
  const float *dK, *dV, *kraw, *h, *act;
  float* part;                            // [4][B][d] partial sums of the split products (RM_PAIR, RM_UP), summed by the next step
  float *dkraw, *dr, *Gz, *dpre, *du, *dh, *dc;
  SyncArea* sync;                         // step timers of instrumented builds
};
inline int rowmat_tasks(const RowmatParams& p, int rb) { return (p.Ncols / p.cols) * ((p.B + rb - 1) / rb) * p.nsplit; }

// One task: `cols` columns of the product for four sequences and one part of a split contraction.  All threads of the CTA.
// Task index t = ((cy * nx) + cx) * nsplit + sp.
// `wslice` (optional): this task's part of the weight matrix already in shared memory, [Kin][cols] -- the cooperative
// kernel keeps it there for all positions of a leaf.
template <typename T, bool COOP, int RB>
__device__ void rowmat_body(const RowmatParams& p, int t, float* smem, const T* wslice = nullptr) {
  const int nx = p.Ncols / p.cols;
  const int sp = t % p.nsplit, cx = (t / p.nsplit) % nx, cy = t / (p.nsplit * nx);
  const int d = p.d;
  const int Kin = p.mode == RM_UP ? p.K / p.nsplit : p.K;   // input entries per row this task needs
  const int k_base = p.mode == RM_UP ? sp * Kin : 0;
  float* in = smem;                                         // [Kin][4] the product's input rows, transposed
  float* st1 = in + (size_t)Kin * RB;              // [Kin][4] staging (u of the RMS backward)
  float* st2 = st1 + (size_t)Kin * RB;             // [Kin][4] staging (the term added)
  float* red = p.mode == RM_UP ? st1 : st2 + (size_t)Kin * RB;   // [16 warps][cols][RB] (the W_up step stages nothing)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b0 = cy * RB;
  const bool writer = cx == 0 && sp == 0;
  const T* gain = reinterpret_cast<const T*>(p.gain);
  const long long part_stride = (long long)p.B * d;
  __syncthreads();                                          // shared memory of the previous task is free

  // ---- prologue: the input rows of this task's sequences, transposed into shared memory
  if (p.mode == RM_PAIR) {
    // task 0: qkRMS backward of dK_i through k_i = qkRMS(kraw_i) per head;  task 1: dV_i as it is
    // (loads of a batch first, stores after: the round trips to L2 overlap instead of queueing behind the stores)
    const float* src = sp ? p.dV : p.dK;
    const bool need_u = !sp && p.qk_on;
    for (int base = threadIdx.x; base < RB * d; base += kRmThreads * 8) {
      float v[8], u[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int idx = base + j * kRmThreads, r = idx / d, e = idx - r * d, b = b0 + r;
        v[j] = 0.f; u[j] = 0.f;
        if (idx < RB * d && b < p.B) {
          const long long at = ((long long)p.i * p.B + b) * d + e;
          v[j] = ld_state<COOP>(src + at);
          if (need_u) u[j] = p.kraw[at];
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int idx = base + j * kRmThreads, r = idx / d, e = idx - r * d;
        if (idx < RB * d) { in[e * RB + r] = v[j]; st1[e * RB + r] = u[j]; }
      }
    }
    if (!sp && p.qk_on) {
      __syncthreads();
      const int H = d / kHeadDim;
      for (int task = warp; task < RB * H; task += kRmWarps) {
        const int r = task / H, c0 = (task % H) * kHeadDim, b = b0 + r;
        const int e0 = c0 + lane, e1 = e0 + 32;
        const float dy0 = in[e0 * RB + r], dy1 = in[e1 * RB + r];
        const float u0 = st1[e0 * RB + r], u1 = st1[e1 * RB + r];
        const float g0 = gain_at(gain, e0), g1 = gain_at(gain, e1);
        const float ss = warp_sum(u0 * u0 + u1 * u1), tu = warp_sum(dy0 * g0 * u0 + dy1 * g1 * u1);
        const float inv = rsqrtf(ss / kHeadDim + p.eps), mean = tu * inv / kHeadDim;
        const float o0 = inv * (dy0 * g0 - u0 * inv * mean), o1 = inv * (dy1 * g1 - u1 * inv * mean);
        in[e0 * RB + r] = o0; in[e1 * RB + r] = o1;
        if (writer && b < p.B) {
          const long long at = ((long long)p.i * p.B + b) * d;
          p.dkraw[at + e0] = o0; p.dkraw[at + e1] = o1;
        }
      }
    } else if (writer) {                                    // no qkRMS: dk_raw = dk
      for (int idx = threadIdx.x; idx < RB * d; idx += kRmThreads) {
        const int r = idx / d, e = idx % d, b = b0 + r;
        if (b < p.B) p.dkraw[((long long)p.i * p.B + b) * d + e] = in[e * RB + r];
      }
    }
  } else if (p.mode == RM_UP) {
    for (int base = threadIdx.x; base < RB * Kin; base += kRmThreads * 8) {
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int idx = base + j * kRmThreads, r = idx / Kin, k = idx - r * Kin, b = b0 + r;
        v[j] = (idx < RB * Kin && b < p.B) ? ld_state<COOP>(p.dpre + ((long long)p.i * p.B + b) * p.K + k_base + k) : 0.f;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int idx = base + j * kRmThreads, r = idx / Kin, k = idx - r * Kin;
        if (idx < RB * Kin) in[k * RB + r] = v[j];
      }
    }
  } else {
    // RM_DOWN: Gz = dz_i + RMS backward of dr_i through RMS(z_i);  RM_OUT: dh = Gz_i + RMS backward of du_i through RMS(h_i),
    // dr_i (du_i) being the sum of the previous step's partial products.  Four warps per row, a quarter of the row each.
    const T* zT = reinterpret_cast<const T*>(p.z);
    constexpr int WPR = kRmWarps / RB;                       // warps per row
    const int r = warp / WPR, quarter = warp % WPR, b = b0 + r;
    const bool live = b < p.B;
    const int e_lo = quarter * (d / WPR), e_hi = e_lo + d / WPR;
    const long long at = ((long long)p.i * p.B + (live ? b : 0)) * d;
    const float* pin = p.part + (long long)(live ? b : 0) * d;
    const T* zr = zT + (long long)(live ? b : 0) * p.z_bs + (long long)p.i * p.z_ts;
    const float* dzr = p.dz + (long long)(live ? b : 0) * p.dz_bs + (long long)p.i * p.dz_ts;
    float* total = (p.mode == RM_DOWN ? p.dr : p.du) + at;   // the summed partials, kept for the gain gradients
    float ss = 0.f, tu = 0.f;
    for (int base = e_lo; base < e_hi; base += 256) {
      float dyv[8], uv[8], av[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + lane + 32 * u;
        dyv[u] = 0.f; uv[u] = 0.f; av[u] = 0.f;
        float pv[4] = {0.f, 0.f, 0.f, 0.f};
        if (e < e_hi && live) {
#pragma unroll
          for (int m = 0; m < 4; ++m)
            if (m < p.n_in) pv[m] = ld_state<COOP>(pin + m * part_stride + e);
          if (p.norm_on) uv[u] = p.mode == RM_DOWN ? to_f(zr[e]) : p.h[at + e];
          av[u] = p.mode == RM_DOWN ? dzr[e] : ld_state<COOP>(p.Gz + at + e);
        }
        dyv[u] = ((pv[0] + pv[1]) + pv[2]) + pv[3];
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + lane + 32 * u;
        if (e < e_hi) {
          if (writer && live) total[e] = dyv[u];
          const float tg = p.norm_on ? dyv[u] * gain_at(gain, e) : dyv[u];
          ss = fmaf(uv[u], uv[u], ss);
          tu = fmaf(tg, uv[u], tu);
          in[e * RB + r] = tg; st1[e * RB + r] = uv[u]; st2[e * RB + r] = av[u];
        }
      }
    }
    ss = warp_sum(ss); tu = warp_sum(tu);
    if (lane == 0) { red[warp * 2] = ss; red[warp * 2 + 1] = tu; }
    __syncthreads();
    ss = 0.f; tu = 0.f;
#pragma unroll
    for (int w = 0; w < WPR; ++w) { ss += red[(r * WPR + w) * 2]; tu += red[(r * WPR + w) * 2 + 1]; }
    const float inv = rsqrtf(ss / d + p.eps), mean = tu * inv / d;
    float* keep = (p.mode == RM_DOWN ? p.Gz : p.dh) + at;
    for (int e = e_lo + lane; e < e_hi; e += 32) {
      const float tg = in[e * RB + r];
      const float du = p.norm_on ? inv * (tg - st1[e * RB + r] * inv * mean) : tg;
      const float val = live ? st2[e * RB + r] + du : 0.f;
      in[e * RB + r] = val;
      if (writer && live) keep[e] = val;
    }
  }
  __syncthreads();

  // ---- product: a warp's lanes = (32 / ncq) rows of W x ncq groups of 4 columns
  const int ncq = p.cols / 4;
  const int kq = lane / ncq, cq = lane % ncq, krows = 32 / ncq;
  const int n0 = cx * p.cols + 4 * cq;
  const T* W = wslice ? wslice + 4 * cq
                      : reinterpret_cast<const T*>(p.mode == RM_PAIR && sp ? p.W2 : p.W1) + (long long)k_base * p.Ncols + n0;
  const long long wstride = wslice ? p.cols : p.Ncols;
  float acc[RB][4] = {};
#pragma unroll 8
  for (int k = warp * krows + kq; k < Kin; k += kRmWarps * krows) {
    Vec4<T> wv;
    wv.v = *reinterpret_cast<const decltype(wv.v)*>(W + (long long)k * wstride);
    float wf[4];
    wv.to_float(wf);
    float av[RB];
#pragma unroll
    for (int r4 = 0; r4 < RB / 4; ++r4) {
      const float4 a4 = *reinterpret_cast<const float4*>(in + (size_t)k * RB + 4 * r4);
      av[4 * r4] = a4.x; av[4 * r4 + 1] = a4.y; av[4 * r4 + 2] = a4.z; av[4 * r4 + 3] = a4.w;
    }
#pragma unroll
    for (int r = 0; r < RB; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], wf[c], acc[r][c]);
  }
#pragma unroll
  for (int r = 0; r < RB; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float v = acc[r][c];
      if (ncq <= 4) v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      if (kq == 0) red[(warp * p.cols + 4 * cq + c) * RB + r] = v;
    }
  __syncthreads();
  if (threadIdx.x < p.cols * RB) {
    const int col = threadIdx.x / RB, r = threadIdx.x % RB, b = b0 + r;
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kRmWarps; ++w) sum += red[(w * p.cols + col) * RB + r];
    if (b < p.B) {
      const int n = cx * p.cols + col;
      sum *= p.alpha;
      if (p.mode == RM_PAIR || p.mode == RM_UP) p.part[sp * part_stride + (long long)b * d + n] = sum;
      else {
        const long long at = ((long long)p.i * p.B + b) * p.Ncols + n;
        if (p.mode == RM_DOWN) p.dpre[at] = sum * gelu_grad_f(p.act[at]);
        else p.dc[at] = sum;
      }
    }
  }
}

template <typename T, int RB>
__global__ void __launch_bounds__(kRmThreads) rowmat_kernel(const RowmatParams p) {
  grid_dep_sync();
  extern __shared__ __align__(16) float smem[];
  rowmat_body<T, false, RB>(p, blockIdx.x, smem);
}

// shared memory of a task: three [K][4] arrays and the reduction area
size_t rowmat_smem(int d, int k_up, int cols, int rb) {
  const size_t in = (size_t)(3 * d > k_up ? 3 * d : k_up) * rb;
  return (in + (size_t)kRmWarps * cols * rb) * sizeof(float);
}

// The reverse loop over one leaf [s0, e0) as ONE cooperative kernel: the five steps of a position separated by grid
// barriers instead of kernel boundaries.  Every wait is bounded (grid_barrier); when one runs out the kernel returns.
struct LoopParams {
  const void *Wk, *Wv, *Wdn, *Wup, *Wo, *g_k, *g_kv, *g_mlp;
  int z_norm, pre, qk;
  int cols_pair, cols_down, cols_up, cols_out, up_split;   // task shapes: columns per task of each step, parts of the W_up contraction
  int resident;                           // 1: every step has at most one task per CTA and its weight slices fit: keep them in shared memory
  unsigned stage_bytes;                   // shared memory of the staging areas (the slices follow)
  float alpha;
  int s0, e0;
  unsigned bar_base;
  SyncArea* sync;
};
constexpr int kLoopBarriersPerPosition = 5;

template <typename T, int RB>
__global__ void __launch_bounds__(kRmThreads, 1) bwd_loop_kernel(RowmatParams p, const LoopParams lp, const AttnBufs a) {
  extern __shared__ __align__(16) float smem[];
  __shared__ int s_flag;
  unsigned target = lp.bar_base;
  const int chunks = (p.B + RB - 1) / RB;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  p.qk_on = lp.qk;
  // weight slices of this CTA's four tasks, resident for the whole leaf
  const T* slice[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  if (lp.resident) {
    T* wsm = reinterpret_cast<T*>(reinterpret_cast<unsigned char*>(smem) + lp.stage_bytes);
    auto stage = [&](int mode, int K, int Ncols, const void* W1, const void* W2, int cols, int nsplit) {
      const int nx = Ncols / cols, tasks = nx * chunks * nsplit, t = blockIdx.x;
      const int Kin = mode == RM_UP ? K / nsplit : K;
      if (t < tasks) {
        const int sp = t % nsplit, cx = (t / nsplit) % nx;
        const T* src = reinterpret_cast<const T*>(mode == RM_PAIR && sp ? W2 : W1) + (long long)(mode == RM_UP ? sp * Kin : 0) * Ncols + cx * cols;
        const int quads = cols / 4;
        for (int idx = threadIdx.x; idx < Kin * quads; idx += kRmThreads) {
          const int k = idx / quads, c4 = idx - k * quads;
          Vec4<T> v;
          v.v = *reinterpret_cast<const decltype(v.v)*>(src + (long long)k * Ncols + 4 * c4);
          *reinterpret_cast<decltype(v.v)*>(wsm + (size_t)k * cols + 4 * c4) = v.v;
        }
        slice[mode] = wsm;
      }
      wsm += (size_t)Kin * cols;                              // every CTA advances alike: the layout is fixed
    };
    stage(RM_PAIR, p.d, p.d, lp.Wk, lp.Wv, lp.cols_pair, 2);
    stage(RM_DOWN, p.d, p.dff, lp.Wdn, nullptr, lp.cols_down, 1);
    stage(RM_UP, p.dff, p.d, lp.Wup, nullptr, lp.cols_up, lp.up_split);
    stage(RM_OUT, p.d, p.d, lp.Wo, nullptr, lp.cols_out, 1);
    __syncthreads();
  }
  auto phase = [&](int mode, int K, int Ncols, const void* W1, const void* W2, const void* gain, int norm_on, float al, int cols,
                   int nsplit, int n_in) {
    p.mode = mode; p.K = K; p.Ncols = Ncols; p.W1 = W1; p.W2 = W2; p.gain = gain; p.norm_on = norm_on; p.alpha = al;
    p.cols = cols; p.nsplit = nsplit; p.n_in = n_in;
    const int tasks = (Ncols / cols) * chunks * nsplit;
    for (int t = blockIdx.x; t < tasks; t += gridDim.x) rowmat_body<T, true, RB>(p, t, smem, slice[mode]);
  };
  // The rows of the next position that nobody has touched since the sweep (dz, z, h, k_raw, W_up u) would each cost a trip
  // to HBM in the middle of a step: the last CTA (never the busiest) asks L2 for them one position ahead.
  auto warm = [&](int pos) {
    if (blockIdx.x != gridDim.x - 1 || pos < 0) return;
    const T* zT = reinterpret_cast<const T*>(p.z);
    for (int b = 0; b < p.B; ++b) {
      const long long at = ((long long)pos * p.B + b) * p.d;
      const int lines_d = p.d / 32, lines_f = p.dff / 32;       // 128-byte lines of fp32 rows
      for (int l = threadIdx.x; l < 3 * lines_d + lines_f + lines_d / 2 + 1; l += kRmThreads) {
        const void* ptr;
        if (l < lines_d) ptr = p.dz + (long long)b * p.dz_bs + (long long)pos * p.dz_ts + 32 * l;
        else if (l < 2 * lines_d) ptr = p.h + at + 32 * (l - lines_d);
        else if (l < 3 * lines_d) ptr = p.kraw + at + 32 * (l - 2 * lines_d);
        else if (l < 3 * lines_d + lines_f) ptr = p.act + ((long long)pos * p.B + b) * p.dff + 32 * (l - 3 * lines_d);
        else {
          const int off = 64 * (l - 3 * lines_d - lines_f);     // 128-byte lines of the storage-type row of z (at most d entries)
          ptr = zT + (long long)b * p.z_bs + (long long)pos * p.z_ts + (off < p.d ? off : 0);
        }
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
      }
    }
  };
  warm(lp.e0 - 1);
  for (int i = lp.e0 - 1; i >= lp.s0; --i) {
    p.i = i;
    warm(i - 1);
    phase(RM_PAIR, p.d, p.d, lp.Wk, lp.Wv, lp.g_k, 0, 1.f, lp.cols_pair, 2, 0);
    if (!grid_barrier(lp.sync, target, gridDim.x, &s_flag)) return;
    phase(RM_DOWN, p.d, p.dff, lp.Wdn, nullptr, lp.g_kv, lp.z_norm, lp.alpha, lp.cols_down, 1, 2);
    if (!grid_barrier(lp.sync, target, gridDim.x, &s_flag)) return;
    phase(RM_UP, p.dff, p.d, lp.Wup, nullptr, nullptr, 0, 1.f, lp.cols_up, lp.up_split, 0);
    if (!grid_barrier(lp.sync, target, gridDim.x, &s_flag)) return;
    phase(RM_OUT, p.d, p.d, lp.Wo, nullptr, lp.g_mlp, lp.pre, lp.alpha, lp.cols_out, 1, lp.up_split);
    if (!grid_barrier(lp.sync, target, gridDim.x, &s_flag)) return;
    const int tasks = (i - lp.s0 + 1) * a.B * a.H;
    for (int t = blockIdx.x * kRmWarps + warp; t < tasks; t += gridDim.x * kRmWarps)
      attn_self_task<true>(a, i, lp.s0 + t / (a.B * a.H), (t / a.H) % a.B, t % a.H, lane);
    if (!grid_barrier(lp.sync, target, gridDim.x, &s_flag)) return;
  }
}

// ------------------------------------------------------------------------------------------------ workspace
struct BwdLayout {
  size_t sync, n, qraw, ktraw, vt, q, kt, r, kraw, k, v, c, h, u, act, gl, lse, D;
  size_t dK, dV, dkraw, dr, Gz, dpre, du, dh, dc, dq, dkt, dvt, dn, gprod, part, part2, sa, sb, wt, wt5, dzp, qkv16;
  size_t zero_begin, zero_end, total;
};
constexpr int kColParts = 128;
constexpr int kWideLeaf = 16;
constexpr int kWideBatchFrom = 32;      // above this many sequences a step of the reverse loop runs as dense products over the batch

BwdLayout bwd_layout(const rt_config* c, int B, int N) {
  BwdLayout L;
  const size_t d = c->d_model, f = c->d_ff, H = c->n_heads, rows = (size_t)B * N;
  size_t o = 0;
  auto take = [&](size_t floats) { size_t at = o; o += align_up(floats * 4, 256); return at; };
  L.sync = take(sizeof(SyncArea) / 4);
  L.n = take(rows * d); L.qraw = take(rows * d); L.ktraw = take(rows * d); L.vt = take(rows * d);
  L.q = take(rows * d); L.kt = take(rows * d); L.r = take(rows * d); L.kraw = take(rows * d);
  L.k = take(rows * d); L.v = take(rows * d); L.c = take(rows * d); L.h = take(rows * d); L.u = take(rows * d);
  L.act = take(rows * f); L.gl = take(rows * f); L.lse = take(rows * H); L.D = take(rows * H);
  L.zero_begin = o;
  L.dK = take(rows * d); L.dV = take(rows * d);
  L.zero_end = o;
  L.dkraw = take(rows * d); L.dr = take(rows * d); L.Gz = take(rows * d); L.dpre = take(rows * f);
  L.du = take(rows * d); L.dh = take(rows * d); L.dc = take(rows * d); L.dq = take(rows * d);
  L.dkt = take(rows * d); L.dvt = take(rows * d); L.dn = take(rows * d); L.gprod = take(rows * d);
  L.part = take((size_t)kColParts * (d > f ? d : f));
  L.part2 = take((size_t)4 * B * d);
  // wide batches: bf16 transposes of the five matrices of the reverse loop, dL/dz in position-major order
  L.qkv16 = take(3 * rows * d / 2 + 64);                       // bf16 copies of q, k, v for the tile kernels
  L.wt5 = take((3 * d * d + 2 * d * f) / 2 + 64); L.dzp = B > kWideBatchFrom ? take(rows * d) : o;
  // bf16 operands of the tensor-core products (bf16 storage): two [rows, max(d, d_ff)] arrays and one [d, d]
  L.sa = take(rows * (d > f ? d : f) / 2 + 64); L.sb = take(rows * (d > f ? d : f) / 2 + 64); L.wt = take(d * d / 2 + 64);
  L.total = o;
  return L;
}

bool bwd_config_ok(const rt_config* c) {
  if (!c) return false;
  if (c->d_model <= 0 || c->n_heads <= 0 || c->d_ff <= 0 || (long long)c->n_heads * c->head_dim != c->d_model) return false;
  if (c->dtype != RT_F32 && c->dtype != RT_BF16) return false;
  if (!(c->rms_eps >= 0.f) || !isfinite(c->softmax_scale) || !isfinite(c->residual_scale)) return false;
  if (c->norm_flags & ~(RT_NORM_PRE | RT_NORM_QK | RT_NORM_SKIP_Z)) return false;
  if (c->flags & ~RT_FLAG_BACKWARD_STEP_LAUNCHES) return false;
  return true;
}

#define RT_TRY(...) do { if ((__VA_ARGS__) != cudaSuccess) return RT_ERR_CUDA; } while (0)

template <typename T>
rt_status backward_impl(const rt_config* c, const rt_layer_weights* w, const T* x, const T* z, const float* dz, int B, int N,
                        float* dx, const rt_layer_grads* gr, unsigned char* ws, cudaStream_t s) {
  const BwdLayout L = bwd_layout(c, B, N);
  const int d = c->d_model, f = c->d_ff, H = c->n_heads;
  const long long rows = (long long)B * N;
  const long long xbs = (long long)N * d, xts = d;             // [B, N, d]
  const long long pbs = d, pts = (long long)B * d;             // position-major fp32 [rows, d] seen as (b, i)
  const bool pre = (c->norm_flags & RT_NORM_PRE) != 0, qk = (c->norm_flags & RT_NORM_QK) != 0;
  const bool z_norm = pre && !(c->norm_flags & RT_NORM_SKIP_Z);
  const float eps = c->rms_eps, alpha = c->residual_scale;
  auto F = [&](size_t off) { return reinterpret_cast<float*>(ws + off); };
  const T *Wq = (const T*)w->w_q, *Wk = (const T*)w->w_k, *Wv = (const T*)w->w_v, *Wo = (const T*)w->w_o;
  const T *Wup = (const T*)w->w_up, *Wdn = (const T*)w->w_down;
  const T *g_attn = (const T*)w->g_attn, *g_mlp = (const T*)w->g_mlp, *g_q = (const T*)w->g_q, *g_k = (const T*)w->g_k;
  const T* g_kv = (const T*)(w->g_kv ? w->g_kv : w->g_attn);
  const int tpb = 256;
  auto warps_grid = [&](long long warps) { return (unsigned)((warps * 32 + tpb - 1) / tpb); };
  auto elems_grid = [&](long long n) { return (unsigned)((n + tpb - 1) / tpb); };

  // Products over all rows.  bf16 storage with tile-friendly widths: tensor cores (dense_tc_kernel) on bf16 copies of
  // the operands, fp32 accumulation and fp32 results; otherwise the fp32 product above.
  constexpr bool kBf16 = sizeof(T) == 2;
  const bool tc = kBf16 && d % 128 == 0 && f % 128 == 0;
  const bool tc_w = tc && rows % 64 == 0;                       // dW = dY^T X contracts over the rows
  SyncArea* sync = reinterpret_cast<SyncArea*>(ws + L.sync);
  __nv_bfloat16* SA = reinterpret_cast<__nv_bfloat16*>(ws + L.sa);
  __nv_bfloat16* SB = reinterpret_cast<__nv_bfloat16*>(ws + L.sb);
  __nv_bfloat16* WT = reinterpret_cast<__nv_bfloat16*>(ws + L.wt);
  auto tc_product = [&](int M, int Nn, int K, const void* A, const void* W, float* out, float al, bool acc, bool chained = false) {
    DenseParams dp;
    memset(&dp, 0, sizeof(dp));
    dp.M = M; dp.N = Nn; dp.K = K; dp.B = 1; dp.A = A; dp.W = W; dp.epi = DENSE_F32; dp.alpha = al; dp.accumulate = acc ? 1 : 0;
    dp.h = out; dp.chained = chained ? 1 : 0;
    if (chained) { dp.partial = F(L.gprod); dp.partial_bytes = (size_t)rows * d * sizeof(float); }   // few rows: split contraction
    return dense_launch(RT_BF16, dp, sync, s);
  };
  auto to_bf16 = [&](const float* in, __nv_bfloat16* out, long long n) {
    to_bf16_kernel<<<elems_grid((n + 3) / 4), tpb, 0, s>>>(in, out, n);
  };
  auto transpose_f = [&](const float* in, long long R, int C, __nv_bfloat16* out) {
    transpose_bf16_kernel<float><<<dim3(ceil_div(C, 32), (unsigned)((R + 31) / 32)), dim3(32, 8), 0, s>>>(in, R, C, out);
  };
  const float* sa_holds = nullptr;                               // which array SA currently holds as a plain bf16 copy
  // out[rows, n_out] = A[rows, k] W[n_out, k]^T  (a product of the forward pass)
  auto fwd_product = [&](const float* A, int k, const T* W, int n_out, float* out) -> cudaError_t {
    if (!tc) return gemm<float, T>((int)rows, n_out, k, A, k, 1, W, 1, k, out, n_out, 1.f, false, s);
    if (sa_holds != A) { to_bf16(A, SA, rows * k); sa_holds = A; }
    return tc_product((int)rows, n_out, k, SA, W, out, 1.f, false);
  };
  // out[rows, n_in] (+)= dY[rows, n_out] W[n_out, n_in]  (gradient of a product's input)
  auto dgrad_product = [&](const float* dY, int n_out, const T* W, int n_in, float* out, bool acc) -> cudaError_t {
    if (!tc) return gemm<float, T>((int)rows, n_in, n_out, dY, n_out, 1, W, n_in, 1, out, n_in, 1.f, acc, s);
    to_bf16(dY, SA, rows * n_out); sa_holds = nullptr;
    transpose_bf16_kernel<T><<<dim3(ceil_div(n_in, 32), ceil_div(n_out, 32)), dim3(32, 8), 0, s>>>(W, n_out, n_in, WT);
    return tc_product((int)rows, n_in, n_out, SA, WT, out, 1.f, acc);
  };
  RT_TRY(cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s));
  RT_TRY(cudaMemsetAsync(ws + L.zero_begin, 0, L.zero_end - L.zero_begin, s));

  // ---- 1. the parallel sweep: every intermediate of the forward pass from x and z
  AttnBufs ab;
  {
  ProfSpanScope span(s, 0);
  norm_fwd_kernel<T, T><<<warps_grid(rows), tpb, 0, s>>>(x, xbs, xts, B, g_attn, F(L.n), rows, d, d, eps, pre ? 1 : 0);
  RT_TRY(fwd_product(F(L.n), d, Wq, d, F(L.qraw)));
  RT_TRY(fwd_product(F(L.n), d, Wk, d, F(L.ktraw)));
  RT_TRY(fwd_product(F(L.n), d, Wv, d, F(L.vt)));
  norm_fwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.qraw), pbs, pts, B, g_q, F(L.q), rows, d, kHeadDim, eps, qk);
  norm_fwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.ktraw), pbs, pts, B, g_k, F(L.kt), rows, d, kHeadDim, eps, qk);
  norm_fwd_kernel<T, T><<<warps_grid(rows), tpb, 0, s>>>(z, xbs, xts, B, g_kv, F(L.r), rows, d, d, eps, z_norm ? 1 : 0);
  RT_TRY(fwd_product(F(L.r), d, Wk, d, F(L.kraw)));
  RT_TRY(fwd_product(F(L.r), d, Wv, d, F(L.v)));
  norm_fwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.kraw), pbs, pts, B, g_k, F(L.k), rows, d, kHeadDim, eps, qk);
  memset(&ab, 0, sizeof(ab));
  ab.q = F(L.q); ab.k = F(L.k); ab.v = F(L.v); ab.kt = F(L.kt); ab.vt = F(L.vt); ab.lse = F(L.lse); ab.D = F(L.D);
  ab.c = F(L.c); ab.dc = F(L.dc); ab.dK = F(L.dK); ab.dV = F(L.dV); ab.dkt = F(L.dkt); ab.dvt = F(L.dvt); ab.dq = F(L.dq);
  ab.alibi = w->alibi_slopes; ab.scale = c->softmax_scale; ab.scale_log2 = c->softmax_scale * kLog2e;
  ab.B = B; ab.H = H; ab.d = d; ab.N = N;
  if (tc) {
    // running softmax state in place of (c, lse, D): seed, the forward pass's tile kernels, finish
    float *st_o = F(L.c), *st_m = F(L.lse), *st_l = F(L.D);
    __nv_bfloat16* q16 = reinterpret_cast<__nv_bfloat16*>(ws + L.qkv16);
    __nv_bfloat16 *k16 = q16 + rows * d, *v16 = k16 + rows * d;
    to_bf16(F(L.q), q16, rows * d); to_bf16(F(L.k), k16, rows * d); to_bf16(F(L.v), v16, rows * d);
    stats_seed_kernel<<<warps_grid(rows * H), tpb, 0, s>>>(ab, st_o, st_m, st_l);
    TileParams tp;
    memset(&tp, 0, sizeof(tp));
    tp.B = B; tp.d = d; tp.H = H; tp.scale_log2 = ab.scale_log2; tp.alibi = w->alibi_slopes;
    tp.q = q16; tp.k_cache = k16; tp.v_cache = v16; tp.st_o = st_o; tp.st_m = st_m; tp.st_l = st_l;
    tp.rows_q = N; tp.rows_kv = N; tp.sync = sync; tp.q_limit = N;
    const int Lb = 128;                                         // diagonal blocks under the causal mask, then Algorithm 1's levels
    const int full = N / Lb;
    tp.causal = 1;
    if (N % Lb == 0 && N >= 4 * Lb) {
      // whole blocks: every query's causal prefix in one launch (a CTA walks over the key blocks up to its own query tile)
      tp.q0 = 0; tp.q1 = N; tp.k0 = 0; tp.k1 = N; tp.causal_full = 1;
      RT_TRY(tile_launch(RT_BF16, tp, s));
      tp.causal_full = 0;
    } else {
      if (full > 0) {
        tp.q0 = 0; tp.q1 = Lb; tp.k0 = 0; tp.k1 = Lb; tp.batch = full; tp.batch_stride = Lb;
        RT_TRY(tile_launch(RT_BF16, tp, s));
      }
      if (full * Lb < N) {
        tp.q0 = full * Lb; tp.q1 = N; tp.k0 = full * Lb; tp.k1 = N; tp.batch = 1; tp.batch_stride = 0;
        RT_TRY(tile_simt_launch(RT_BF16, tp, s));
      }
      tp.causal = 0;
      for (long long P = Lb; P < N; P *= 2) {
        tp.q0 = (int)P; tp.q1 = (int)(2 * P); tp.k0 = 0; tp.k1 = (int)P;
        tp.batch = (int)((N - P + 2 * P - 1) / (2 * P)); tp.batch_stride = (int)(2 * P);
        RT_TRY(tile_launch(RT_BF16, tp, s));
      }
    }
    stats_finish_kernel<<<warps_grid(rows * H), tpb, 0, s>>>(ab, st_o, st_m, st_l);
  } else {
    attn_stats_kernel<<<warps_grid((long long)((N + 3) / 4) * B * H), tpb, 0, s>>>(ab);
  }
  RT_TRY(fwd_product(F(L.c), d, Wo, d, F(L.dn)));                     // a = W_o c (dn as scratch)
  residual_kernel<T><<<elems_grid(rows * d), tpb, 0, s>>>(x, xbs, xts, B, F(L.dn), alpha, F(L.h), rows, d);
  norm_fwd_kernel<float, T><<<warps_grid(rows), tpb, 0, s>>>(F(L.h), pbs, pts, B, g_mlp, F(L.u), rows, d, d, eps, pre ? 1 : 0);
  RT_TRY(fwd_product(F(L.u), d, Wup, f, F(L.act)));
  gelu_kernel<<<elems_grid(rows * f), tpb, 0, s>>>(F(L.act), F(L.gl), rows * f);
  RT_TRY(cudaGetLastError());
  }

  // ---- 2. the reverse loop: only d(k_j, v_j) accumulate here
  RowmatParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.B = B; rp.d = d; rp.dff = f; rp.eps = eps;
  rp.z = z; rp.z_bs = xbs; rp.z_ts = xts; rp.dz = dz; rp.dz_bs = xbs; rp.dz_ts = xts;
  rp.dK = F(L.dK); rp.dV = F(L.dV); rp.kraw = F(L.kraw); rp.h = F(L.h); rp.act = F(L.act);
  rp.dkraw = F(L.dkraw); rp.dr = F(L.dr); rp.Gz = F(L.Gz); rp.dpre = F(L.dpre); rp.du = F(L.du); rp.dh = F(L.dh); rp.dc = F(L.dc);
  int dev = 0, sms = 0, per_sm = 0, coop = 0;
  RT_TRY(cudaGetDevice(&dev));
  RT_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  RT_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
  const int rb = 4;                                              // sequences per task (8 per task measured slower: B = 8, d = 1024: 69 vs 59 us per position)
  const int chunks = ceil_div(B, rb);
  // task shapes: the W_up contraction in as many parts (of whole 128-row strides) as keep the grid busy once; the
  // W_down step with 32 columns per task when 16 would need more than one round of the grid
  // 16 columns per task, 32 where 16 would need more than one round of the grid (each task repeats the step's prologue)
  const int cols_pair = (d / 16) * chunks * 2 > sms ? 32 : 16;
  const int cols_out = (d / 16) * chunks > sms ? 32 : 16;
  const int cols_down = (f / 16) * chunks > sms ? 32 : 16;
  int up_split = 1, cols_up = (d / 16) * chunks > sms ? 32 : 16;
  for (int c = 4; c >= 2; --c)
    if (f % (c * 128) == 0 && (d / cols_up) * chunks * c <= sms) { up_split = c; break; }
  rp.part = F(L.part2); rp.sync = reinterpret_cast<SyncArea*>(ws + L.sync);
  const size_t smem_max = rowmat_smem(d, f / up_split, 32, rb);
  if (smem_max > 200 * 1024) return RT_ERR_UNSUPPORTED;
  const void* step_fn = reinterpret_cast<const void*>(&rowmat_kernel<T, 4>);
  const void* loop_fn = reinterpret_cast<const void*>(&bwd_loop_kernel<T, 4>);
  RT_TRY(cudaFuncSetAttribute(step_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
  auto rowmat = [&](int mode, int i, int K, int Ncols, const void* W1, const void* W2, const void* gain, int norm_on, float al, int cols,
                    int nsplit, int n_in) {
    rp.mode = mode; rp.i = i; rp.K = K; rp.Ncols = Ncols; rp.W1 = W1; rp.W2 = W2; rp.gain = gain;
    rp.norm_on = norm_on; rp.qk_on = qk ? 1 : 0; rp.alpha = al; rp.cols = cols; rp.nsplit = nsplit; rp.n_in = n_in;
    const dim3 grid(rowmat_tasks(rp, rb)), block(kRmThreads);
    return launch_chained(rowmat_kernel<T, 4>, grid, block, smem_max, s, true, rp);
  };
  RT_TRY(cudaFuncSetAttribute(loop_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
  RT_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bwd_loop_kernel<T, 4>, kRmThreads, smem_max));
  // RT_FLAG_BACKWARD_STEP_LAUNCHES in the configuration forces the one-launch-per-step form (what a device without
  // cooperative launch gets; the tests run both forms)
  bool use_coop = coop && per_sm >= 1 && !(c->flags & RT_FLAG_BACKWARD_STEP_LAUNCHES);
  // weight slices resident in shared memory when every step has at most one task per CTA and they fit beside the staging
  const size_t slice_bytes = ((size_t)d * cols_pair + (size_t)d * cols_down + (size_t)(f / up_split) * cols_up + (size_t)d * cols_out) * sizeof(T);
  const bool one_task = (d / cols_pair) * chunks * 2 <= sms && (f / cols_down) * chunks <= sms && (d / cols_up) * chunks * up_split <= sms &&
                        (d / cols_out) * chunks <= sms;
  size_t loop_smem = smem_max;
  bool resident = false;
  if (use_coop && one_task && smem_max + slice_bytes <= 220 * 1024) {
    int per_sm_res = 0;
    RT_TRY(cudaFuncSetAttribute(loop_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem_max + slice_bytes)));
    RT_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_res, bwd_loop_kernel<T, 4>, kRmThreads, smem_max + slice_bytes));
    if (per_sm_res >= 1) { resident = true; loop_smem = smem_max + slice_bytes; }
  }
  LoopParams lp;
  memset(&lp, 0, sizeof(lp));
  lp.Wk = Wk; lp.Wv = Wv; lp.Wdn = Wdn; lp.Wup = Wup; lp.Wo = Wo; lp.g_k = g_k; lp.g_kv = g_kv; lp.g_mlp = g_mlp;
  lp.z_norm = z_norm ? 1 : 0; lp.pre = pre ? 1 : 0; lp.qk = qk ? 1 : 0; lp.alpha = alpha;
  lp.cols_pair = cols_pair; lp.cols_down = cols_down; lp.cols_up = cols_up; lp.cols_out = cols_out; lp.up_split = up_split;
  lp.resident = resident ? 1 : 0; lp.stage_bytes = (unsigned)smem_max;
  lp.sync = reinterpret_cast<SyncArea*>(ws + L.sync);
  unsigned bar_base = 0;
  // leaf of the reverse schedule; wide batches take short leaves (the in-leaf step re-reads and rewrites the fp32
  // pairs of its leaf at every position, the tiles do not)
  const int Lf = B > kWideBatchFrom ? kWideLeaf : 64;
  // Wide batches (the paper's own regime, Sec. 6): a step of the reverse loop is a dense product over the B rows of the
  // position -- tensor cores for bf16 storage -- between small row-wise kernels, instead of tasks of four sequences.
  const bool wide = B > kWideBatchFrom;
  const size_t pos_d = (size_t)B * d, pos_f = (size_t)B * f;
  __nv_bfloat16* WkT = reinterpret_cast<__nv_bfloat16*>(ws + L.wt5);
  __nv_bfloat16 *WvT = WkT + (size_t)d * d, *WoT = WvT + (size_t)d * d, *WdnT = WoT + (size_t)d * d, *WupT = WdnT + (size_t)d * f;
  if (wide) {
    norm_fwd_kernel<float, T><<<warps_grid(rows), tpb, 0, s>>>(dz, xbs, xts, B, (const T*)nullptr, F(L.dzp), rows, d, d, eps, 0);
    if (tc) {
      auto tr = [&](const T* W, int n_out, int n_in, __nv_bfloat16* out) {
        transpose_bf16_kernel<T><<<dim3(ceil_div(n_in, 32), ceil_div(n_out, 32)), dim3(32, 8), 0, s>>>(W, n_out, n_in, out);
      };
      tr(Wk, d, d, WkT); tr(Wv, d, d, WvT); tr(Wo, d, d, WoT); tr(Wdn, d, f, WdnT); tr(Wup, f, d, WupT);
    }
    RT_TRY(cudaGetLastError());
  }
  // out[B, n_in] (+)= al * dY[B, n_out] W[n_out, n_in] for the rows of one position; A_bf = bf16 copy of dY (scale folded in)
  auto step_product = [&](const float* dY, const __nv_bfloat16* A_bf, int n_out, const T* W, const __nv_bfloat16* Wt, int n_in, float* out,
                          float al, bool acc) -> cudaError_t {
    if (!tc) return gemm<float, T>(B, n_in, n_out, dY, n_out, 1, W, n_in, 1, out, n_in, al, acc, s);
    return tc_product(B, n_in, n_out, A_bf, Wt, out, 1.f, acc, true);
  };
  // The launches of a position are chained (programmatic dependent launches); each producer also leaves the bf16 operand
  // of the product that follows (SA, SB), so a position is eleven launches.
  auto wide_position = [&](int i, int s0) -> rt_status {
    const size_t od = (size_t)i * pos_d, of = (size_t)i * pos_f;
    sa_holds = nullptr;
    const dim3 blk(tpb);
    // dk_raw = qkRMS backward of dk_i;  dr = dk_raw W_k + dv_i W_v
    RT_TRY(launch_chained(norm_bwd_kernel<float, T>, dim3(warps_grid((long long)B * H)), blk, 0, s, true, (const float*)(F(L.dK) + od),
                          (const float*)(F(L.kraw) + od), pbs, pts, B, g_k, (const float*)nullptr, F(L.dkraw) + od, pbs, pts, (float*)nullptr, 0,
                          (long long)B, d, (int)kHeadDim, eps, qk ? 1 : 0, tc ? SA : (__nv_bfloat16*)nullptr, 1.f));
    if (tc) RT_TRY(launch_chained(to_bf16_kernel, dim3(elems_grid((long long)(pos_d + 3) / 4)), blk, 0, s, true, (const float*)(F(L.dV) + od), SB,
                                  (long long)pos_d));
    RT_TRY(step_product(F(L.dkraw) + od, SA, d, Wk, WkT, d, F(L.dr) + od, 1.f, false));
    RT_TRY(step_product(F(L.dV) + od, SB, d, Wv, WvT, d, F(L.dr) + od, 1.f, true));
    // Gz = dz_i + RMS backward of dr;  dpre = (alpha Gz W_down) * GELU'
    RT_TRY(launch_chained(norm_bwd_row_kernel<T, T>, dim3(B), dim3(256), 0, s, true, (const float*)(F(L.dr) + od), z + (size_t)i * xts, xbs, xts, B,
                          g_kv, (const float*)(F(L.dzp) + od), F(L.Gz) + od, d, eps, z_norm ? 1 : 0, tc ? SA : (__nv_bfloat16*)nullptr, alpha));
    RT_TRY(step_product(F(L.Gz) + od, SA, d, Wdn, WdnT, f, F(L.dpre) + of, alpha, false));
    RT_TRY(launch_chained(gelu_bwd_kernel, dim3(elems_grid(((long long)pos_f + 3) / 4)), blk, 0, s, true, F(L.dpre) + of, (const float*)(F(L.act) + of),
                          (long long)pos_f, tc ? SA : (__nv_bfloat16*)nullptr));
    // du = dpre W_up;  dh = Gz + RMS backward of du;  dc = alpha dh W_o
    RT_TRY(step_product(F(L.dpre) + of, SA, f, Wup, WupT, d, F(L.du) + od, 1.f, false));
    RT_TRY(launch_chained(norm_bwd_row_kernel<float, T>, dim3(B), dim3(256), 0, s, true, (const float*)(F(L.du) + od), (const float*)(F(L.h) + od),
                          pbs, pts, B, g_mlp, (const float*)(F(L.Gz) + od), F(L.dh) + od, d, eps, pre ? 1 : 0,
                          tc ? SA : (__nv_bfloat16*)nullptr, alpha));
    RT_TRY(step_product(F(L.dh) + od, SA, d, Wo, WoT, d, F(L.dc) + od, alpha, false));
    // the query's share of the pairs of its own leaf, its temporary pair and D_i
    RT_TRY(launch_chained(attn_self_wide_kernel, dim3(warps_grid((long long)B * H)), blk, 0, s, true, ab, i, s0));
    return RT_OK;
  };
  RT_TRY(cudaFuncSetAttribute(attn_bwd_kv_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairBlockSmem));
  for (int s0 = ((N - 1) / Lf) * Lf; s0 >= 0; s0 -= Lf) {
    const int e0 = s0 + Lf < N ? s0 + Lf : N;
    if (e0 < N) {                                                // Algorithm 1's tile at block end e0, backwards
      const int P = e0 & -e0;
      const int q1 = e0 + P < N ? e0 + P : N;
      ProfSpanScope span(s, 2);
      if (P % kPB == 0 && (long long)B * H <= 65535) {
        RT_TRY(launch_chained(attn_bwd_kv_block_kernel, dim3(P / kPB, B * H), dim3(256), kPairBlockSmem, s, !use_coop && !wide, ab, e0, q1,
                              e0 - P, e0));
      } else {
        RT_TRY(launch_chained(attn_bwd_kv_tile_kernel, dim3(warps_grid((long long)P * B * H)), dim3(tpb), 0, s, !use_coop && !wide, ab,
                              e0, q1, e0 - P, e0));
      }
    }
    ProfSpanScope span(s, 1);
    if (wide) {
      for (int i = e0 - 1; i >= s0; --i) {
        const rt_status st = wide_position(i, s0);
        if (st != RT_OK) return st;
      }
      continue;
    }
    if (use_coop) {
      lp.s0 = s0; lp.e0 = e0; lp.bar_base = bar_base;
      void* args[] = {(void*)&rp, (void*)&lp, (void*)&ab};
      RT_TRY(cudaLaunchCooperativeKernel(loop_fn, dim3(sms), dim3(kRmThreads), args, loop_smem, s));
      bar_base += (unsigned)(e0 - s0) * kLoopBarriersPerPosition * (unsigned)sms;
      continue;
    }
    for (int i = e0 - 1; i >= s0; --i) {
      RT_TRY(rowmat(RM_PAIR, i, d, d, Wk, Wv, g_k, 0, 1.f, cols_pair, 2, 0));
      RT_TRY(rowmat(RM_DOWN, i, d, f, Wdn, nullptr, g_kv, z_norm ? 1 : 0, alpha, cols_down, 1, 2));
      RT_TRY(rowmat(RM_UP, i, f, d, Wup, nullptr, nullptr, 0, 1.f, cols_up, up_split, 0));
      RT_TRY(rowmat(RM_OUT, i, d, d, Wo, nullptr, g_mlp, pre ? 1 : 0, alpha, cols_out, 1, up_split));
      RT_TRY(launch_chained(attn_bwd_kv_kernel, dim3(warps_grid((long long)(i - s0 + 1) * B * H)), dim3(tpb), 0, s, true, ab, i, s0));
    }
  }

  // ---- 3. everything else over all rows at once
  ProfSpanScope span(s, 3);
  if ((long long)B * H <= 65535) {
    RT_TRY(cudaFuncSetAttribute(attn_bwd_q_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairBlockSmemQ));
    attn_bwd_q_block_kernel<<<dim3(ceil_div(N, kPB), B * H), 256, kPairBlockSmemQ, s>>>(ab);
  } else {
    attn_bwd_q_kernel<<<warps_grid((long long)((N + 3) / 4) * B * H), tpb, 0, s>>>(ab);
  }
  float* gprod = F(L.gprod);
  float* part = F(L.part);
  auto col_sum = [&](const float* a, int width, float* out, bool acc) {
    col_partial_kernel<<<dim3(ceil_div(width, 128), kColParts), 128, 0, s>>>(a, rows, width, part, kColParts);
    col_final_kernel<<<ceil_div(width, 128), 128, 0, s>>>(part, kColParts, width, out, acc ? 1 : 0);
  };
  // qkRMS backward of dq and of the temporary keys (in place), and their gain products
  const bool want_gq = gr->g_q && w->g_q && qk, want_gk = gr->g_k && w->g_k && qk;
  norm_bwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.dq), F(L.qraw), pbs, pts, B, g_q, nullptr, F(L.dq), pbs, pts,
                                                                 want_gq ? gprod : nullptr, 0, rows, d, kHeadDim, eps, qk);
  if (want_gq) col_sum(gprod, d, gr->g_q, false);
  else if (gr->g_q) RT_TRY(cudaMemsetAsync(gr->g_q, 0, (size_t)d * 4, s));
  norm_bwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.dkt), F(L.ktraw), pbs, pts, B, g_k, nullptr, F(L.dkt), pbs, pts,
                                                                 want_gk ? gprod : nullptr, 0, rows, d, kHeadDim, eps, qk);
  if (want_gk) {
    norm_bwd_kernel<float, T><<<warps_grid(rows * H), tpb, 0, s>>>(F(L.dK), F(L.kraw), pbs, pts, B, g_k, nullptr, nullptr, pbs, pts,
                                                                   gprod, 1, rows, d, kHeadDim, eps, qk);
    col_sum(gprod, d, gr->g_k, false);
  } else if (gr->g_k) RT_TRY(cudaMemsetAsync(gr->g_k, 0, (size_t)d * 4, s));
  // dn = dqraw W_q + dktraw W_k + dvt W_v;  dx = dh + RMS backward of dn through RMS(x)
  RT_TRY(dgrad_product(F(L.dq), d, Wq, d, F(L.dn), false));
  RT_TRY(dgrad_product(F(L.dkt), d, Wk, d, F(L.dn), true));
  RT_TRY(dgrad_product(F(L.dvt), d, Wv, d, F(L.dn), true));
  const bool want_ga = gr->g_attn && w->g_attn && pre;
  norm_bwd_kernel<T, T><<<warps_grid(rows), tpb, 0, s>>>(F(L.dn), x, xbs, xts, B, g_attn, F(L.dh), dx, xbs, xts,
                                                         want_ga ? gprod : nullptr, 0, rows, d, d, eps, pre ? 1 : 0);
  // gains of RMS(x) and RMS(z): one array when g_kv is not given (then RMS(z) uses g_attn)
  const bool kv_alias = w->g_kv == nullptr;
  if (want_ga) {
    if (kv_alias && z_norm)
      norm_bwd_kernel<T, T><<<warps_grid(rows), tpb, 0, s>>>(F(L.dr), z, xbs, xts, B, g_kv, nullptr, nullptr, pbs, pts, gprod, 1, rows, d,
                                                             d, eps, 1);
    col_sum(gprod, d, gr->g_attn, false);
  } else if (gr->g_attn) RT_TRY(cudaMemsetAsync(gr->g_attn, 0, (size_t)d * 4, s));
  if (gr->g_kv) {
    if (!kv_alias && z_norm) {
      norm_bwd_kernel<T, T><<<warps_grid(rows), tpb, 0, s>>>(F(L.dr), z, xbs, xts, B, g_kv, nullptr, nullptr, pbs, pts, gprod, 0, rows, d,
                                                             d, eps, 1);
      col_sum(gprod, d, gr->g_kv, false);
    } else RT_TRY(cudaMemsetAsync(gr->g_kv, 0, (size_t)d * 4, s));
  }
  if (gr->g_mlp) {
    if (w->g_mlp && pre) {
      norm_bwd_kernel<float, T><<<warps_grid(rows), tpb, 0, s>>>(F(L.du), F(L.h), pbs, pts, B, g_mlp, nullptr, nullptr, pbs, pts, gprod, 0,
                                                                 rows, d, d, eps, 1);
      col_sum(gprod, d, gr->g_mlp, false);
    } else RT_TRY(cudaMemsetAsync(gr->g_mlp, 0, (size_t)d * 4, s));
  }
  // parameter matrices: dW[o, i] = sum_rows dY[row, o] X[row, i]
  const float* sb_holds = nullptr;                               // which array SB currently holds transposed
  auto wgrad = [&](float* out, const float* dY, int n_out, const float* X, int n_in, float al, bool acc) -> cudaError_t {
    if (!tc_w) return gemm<float, float>(n_out, n_in, (int)rows, dY, 1, n_out, X, n_in, 1, out, n_in, al, acc, s);
    transpose_f(dY, rows, n_out, SA); sa_holds = nullptr;
    if (sb_holds != X) { transpose_f(X, rows, n_in, SB); sb_holds = X; }
    return tc_product(n_out, n_in, (int)rows, SA, SB, out, al, acc);
  };
  if (gr->w_k) RT_TRY(wgrad(gr->w_k, F(L.dkraw), d, F(L.r), d, 1.f, false));
  if (gr->w_v) RT_TRY(wgrad(gr->w_v, F(L.dV), d, F(L.r), d, 1.f, false));
  if (gr->w_k) RT_TRY(wgrad(gr->w_k, F(L.dkt), d, F(L.n), d, 1.f, true));
  if (gr->w_v) RT_TRY(wgrad(gr->w_v, F(L.dvt), d, F(L.n), d, 1.f, true));
  if (gr->w_q) RT_TRY(wgrad(gr->w_q, F(L.dq), d, F(L.n), d, 1.f, false));
  if (gr->w_o) RT_TRY(wgrad(gr->w_o, F(L.dh), d, F(L.c), d, alpha, false));
  if (gr->w_up) RT_TRY(wgrad(gr->w_up, F(L.dpre), f, F(L.u), d, 1.f, false));
  if (gr->w_down) RT_TRY(wgrad(gr->w_down, F(L.Gz), d, F(L.gl), f, alpha, false));
  RT_TRY(cudaGetLastError());
  return RT_OK;
}

}  // namespace
}  // namespace rt

extern "C" {

size_t rt_backward_workspace_bytes(const rt_config* cfg, int32_t B, int32_t N) {
  if (!rt::bwd_config_ok(cfg) || B <= 0 || N <= 0) return 0;
  return rt::bwd_layout(cfg, B, N).total;
}

rt_status rt_layer_backward(const rt_config* cfg, const rt_layer_weights* w, const void* x, const void* z, const float* dz,
                            int32_t B, int32_t N, float* dx, const rt_layer_grads* grads, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
  using namespace rt;
  if (!bwd_config_ok(cfg) || B <= 0 || N <= 0 || !workspace || ((uintptr_t)workspace & 15)) return RT_ERR_INVALID_ARG;
  if (cfg->head_dim != kHeadDim || cfg->d_ff % 32 || cfg->recur_block > 1)
    return RT_ERR_UNSUPPORTED;
  if (!w || !w->w_q || !w->w_k || !w->w_v || !w->w_o || !w->w_up || !w->w_down || !x || !z || !dz || !dx || !grads)
    return RT_ERR_INVALID_ARG;
  if (((uintptr_t)x | (uintptr_t)z | (uintptr_t)dz | (uintptr_t)dx) & 15) return RT_ERR_INVALID_ARG;
  {
    const float* gp[] = {grads->w_q, grads->w_k, grads->w_v, grads->w_o, grads->w_up, grads->w_down,
                         grads->g_attn, grads->g_mlp, grads->g_kv, grads->g_q, grads->g_k};
    for (const float* ptr : gp)
      if ((uintptr_t)ptr & 15) return RT_ERR_INVALID_ARG;
  }
  if (workspace_bytes < bwd_layout(cfg, B, N).total) return RT_ERR_WORKSPACE;
  if ((long long)B * N > 0x7fffffffLL / 2) return RT_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (cfg->dtype == RT_BF16)
    return backward_impl<__nv_bfloat16>(cfg, w, (const __nv_bfloat16*)x, (const __nv_bfloat16*)z, dz, B, N, dx, grads,
                                        (unsigned char*)workspace, s);
  return backward_impl<float>(cfg, w, (const float*)x, (const float*)z, dz, B, N, dx, grads, (unsigned char*)workspace, s);
}

}  // extern "C"
