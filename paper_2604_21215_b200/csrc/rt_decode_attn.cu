// Attention of one decode step over the whole cache (bf16 storage): the new position's query of every (sequence, head)
// against the persistent pairs [0, pos), as Algorithm 2 applied to chunks of the cache whose partial states (m, l, o) are
// merged, in chunk order, into the state seeded with the temporary pair (by the attention warps of the leaf kernel that
// runs the token step).  A forward pass is a sequence of such steps (Sec. 5); with a long cache the step is bound by
// streaming K and V once (2 pos B d e bytes per layer).
//
// partial kernel: a CTA takes one chunk of positions of one sequence, a warp one head.  Scores: lane = key (the lane reads
// its key's 128-byte row; the query sits in shared memory, read as broadcasts), no shuffles per product.  Values:
// lane = two dimensions (the warp reads a V row as one coalesced 128-byte line, the key's weight comes by shuffle), so a
// lane keeps two accumulators.  All 40 loads of a group of 32 keys are issued before the first product.
#include <cuda_bf16.h>

#include "rt_kernels.h"

namespace rt {

namespace {

constexpr int kDecWarps = 8;

__device__ __forceinline__ float bf_lo_f(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi_f(unsigned u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kDecWarps * 32, 2) decode_attn_partial_kernel(const DecodeAttnParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = blockIdx.x, b = blockIdx.y, h = blockIdx.z * kDecWarps + warp;
  if (h >= p.H) return;
  const int j0 = chunk * p.chunk, j1 = min(j0 + p.chunk, p.pos);
  float* out = p.part + ((size_t)(b * p.H + h) * p.n_chunks + chunk) * 66;
  if (j0 >= j1) {                                             // (cannot happen with the launcher's chunking; kept for safety)
    if (lane == 0) { out[64] = -INFINITY; out[65] = 0.f; }
    out[2 * lane] = 0.f; out[2 * lane + 1] = 0.f;
    return;
  }
  const __nv_bfloat16* kc = reinterpret_cast<const __nv_bfloat16*>(p.k_cache) + (size_t)b * p.d + h * kHeadDim;
  const __nv_bfloat16* vc = reinterpret_cast<const __nv_bfloat16*>(p.v_cache) + (size_t)b * p.d + h * kHeadDim;
  const size_t row_stride = (size_t)p.B * p.d;                // elements between consecutive positions
  // the query (already normalised by the pre-pass) in shared memory as fp32: every lane multiplies its own key by the
  // same query values, so the reads are broadcasts and the registers stay free for loads in flight
  __shared__ float4 q_s[kDecWarps][kHeadDim / 4];
  {
    const unsigned* qp = reinterpret_cast<const unsigned*>(reinterpret_cast<const __nv_bfloat16*>(p.q) + (size_t)b * p.d + h * kHeadDim);
    const unsigned w = qp[lane];
    reinterpret_cast<float2*>(&q_s[warp][0])[lane] = make_float2(bf_lo_f(w), bf_hi_f(w));
  }
  __syncwarp();
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;
  const size_t vstride = row_stride / 2;                      // 32-bit words between rows
  float m_run = -INFINITY, l_lane = 0.f, o0 = 0.f, o1 = 0.f;
  for (int g0 = j0; g0 < j1; g0 += 32) {
    const int j = g0 + lane;
    const bool valid = j < j1;
    const int jr = valid ? j : j1 - 1;                        // rows read by lanes beyond the chunk (masked below)
    const int n_here = min(32, j1 - g0);
    // all loads of the group first: this lane's key row (128 bytes), and for the values one coalesced 128-byte row per
    // key with lane = dimensions 2 lane, 2 lane + 1
    const uint4* kp = reinterpret_cast<const uint4*>(kc + (size_t)jr * row_stride);
    uint4 kw[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) kw[i] = kp[i];
    const unsigned* vp = reinterpret_cast<const unsigned*>(vc + (size_t)g0 * row_stride) + lane;
    unsigned vw[32];
#pragma unroll
    for (int jj = 0; jj < 32; ++jj) vw[jj] = vp[(size_t)(jj < n_here ? jj : n_here - 1) * vstride];
    // ---- scores: this lane's key against the query ----
    float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float4 qa = q_s[warp][2 * i], qb = q_s[warp][2 * i + 1];
      d0 = fmaf(bf_lo_f(kw[i].x), qa.x, d0); d1 = fmaf(bf_hi_f(kw[i].x), qa.y, d1);
      d2 = fmaf(bf_lo_f(kw[i].y), qa.z, d2); d3 = fmaf(bf_hi_f(kw[i].y), qa.w, d3);
      d0 = fmaf(bf_lo_f(kw[i].z), qb.x, d0); d1 = fmaf(bf_hi_f(kw[i].z), qb.y, d1);
      d2 = fmaf(bf_lo_f(kw[i].w), qb.z, d2); d3 = fmaf(bf_hi_f(kw[i].w), qb.w, d3);
    }
    float s = ((d0 + d1) + (d2 + d3)) * p.scale_log2 - slope_l2 * (float)(p.pos - j);      // ALiBi distance pos - j
    if (!valid) s = -INFINITY;
    // ---- Algorithm 2 with this group of 32 keys as the tile ----
    const float m_new = fmaxf(m_run, warp_max(s));            // finite: the group holds at least one key
    const float corr = ex2f(m_run - m_new);                   // 0 for the first group (m_run = -inf)
    const float pj = valid ? ex2f(s - m_new) : 0.f;
    l_lane = l_lane * corr + pj;
    o0 *= corr; o1 *= corr;
    m_run = m_new;
    // ---- values: the key's weight comes by shuffle (0 for keys beyond the chunk) ----
#pragma unroll
    for (int jj = 0; jj < 32; ++jj) {
      const float w = __shfl_sync(0xffffffffu, pj, jj);
      o0 = fmaf(w, bf_lo_f(vw[jj]), o0);
      o1 = fmaf(w, bf_hi_f(vw[jj]), o1);
    }
  }
  const float l = warp_sum(l_lane);
  *reinterpret_cast<float2*>(out + 2 * lane) = make_float2(o0, o1);
  if (lane == 0) { out[64] = m_run; out[65] = l; }
}

}  // namespace

// Chunking of a cache of `pos` positions: whole groups of 32 keys, at most kDecodeMaxChunks chunks.
int decode_attn_chunk(int pos) {
  int chunk = 64;
  while ((pos + chunk - 1) / chunk > kDecodeMaxChunks) chunk *= 2;
  return chunk;
}

cudaError_t decode_attn_launch(const DecodeAttnParams& p0, int* n_chunks, cudaStream_t s) {
  DecodeAttnParams p = p0;
  *n_chunks = 0;
  if (p.pos <= 0) return cudaSuccess;
  p.chunk = decode_attn_chunk(p.pos);
  p.n_chunks = (p.pos + p.chunk - 1) / p.chunk;
  *n_chunks = p.n_chunks;
  dim3 grid(p.n_chunks, p.B, ceil_div(p.H, kDecWarps));
  decode_attn_partial_kernel<<<grid, kDecWarps * 32, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace rt
