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
constexpr int kDecodeRowsFrom = 2048;            // cache lengths from which the lane = pair kernel streams the cache

int sm_count_cached() {
  thread_local int dev_cached = -1, sms = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev != dev_cached) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) { sms = n; dev_cached = dev; }
  }
  return sms;
}

__device__ __forceinline__ float bf_lo_f(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi_f(unsigned u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kDecWarps * 32) decode_attn_partial_kernel(const DecodeAttnParams p) {
  grid_dep_sync();                                           // the launches of a decode step are chained (programmatic dependent launches)
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


// ---- long caches: lane = (sequence, head) ---------------------------------------------------------------------------
// With many positions per chunk the cache is read fastest when consecutive lanes read consecutive segments of the same
// position-major row: a pair of lanes owns a (sequence, head) pair, a warp reads 2 KB of a K row and 2 KB of a V row per
// key, each lane pair runs Algorithm 2 for its pair key by key (one shuffle per key, no shared memory) with the next
// key's rows in flight while it works on the current one.  A second kernel merges the chunk partials of a pair in parallel.
constexpr int kRowThreads = 256;

__device__ __forceinline__ void load_half(const __nv_bfloat16* p, uint4 (&r)[4]) {
  const uint4* q = reinterpret_cast<const uint4*>(p);
#pragma unroll
  for (int i = 0; i < 4; ++i) r[i] = q[i];
}
__device__ __forceinline__ float dot_half(const uint4 (&k)[4], const uint4 (&q)[4]) {
  float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    d0 = fmaf(bf_lo_f(k[i].x), bf_lo_f(q[i].x), d0); d1 = fmaf(bf_hi_f(k[i].x), bf_hi_f(q[i].x), d1);
    d2 = fmaf(bf_lo_f(k[i].y), bf_lo_f(q[i].y), d2); d3 = fmaf(bf_hi_f(k[i].y), bf_hi_f(q[i].y), d3);
    d0 = fmaf(bf_lo_f(k[i].z), bf_lo_f(q[i].z), d0); d1 = fmaf(bf_hi_f(k[i].z), bf_hi_f(q[i].z), d1);
    d2 = fmaf(bf_lo_f(k[i].w), bf_lo_f(q[i].w), d2); d3 = fmaf(bf_hi_f(k[i].w), bf_hi_f(q[i].w), d3);
  }
  return (d0 + d1) + (d2 + d3);
}

// Two lanes per pair, 32 dimensions (64 bytes of a row) each: half the registers of one lane per pair, so two CTAs share
// an SM and twice as many loads are in flight; the two halves of a logit meet through one shuffle per key.
__global__ void __launch_bounds__(kRowThreads, 2) decode_attn_rows_kernel(const DecodeAttnParams p) {
  grid_dep_sync();                                           // the launches of a decode step are chained (programmatic dependent launches)
  const int seg = blockIdx.y * kRowThreads + threadIdx.x;     // 32-element segment of a row
  const int u = seg >> 1, half = seg & 1;                     // (sequence, head) pair and which half of its 64 dimensions
  const bool live = u < p.B * p.H;
  const int uu = live ? u : 0;                                // lanes beyond the last pair shadow pair 0 (their shuffles are needed)
  const int chunk = blockIdx.x;
  const int j0 = chunk * p.chunk, j1 = min(j0 + p.chunk, p.pos);
  float* out = p.part + ((size_t)uu * p.n_chunks + chunk) * 66;
  const int h = uu % p.H;
  const size_t row_stride = (size_t)p.B * p.d;
  const __nv_bfloat16* kc = reinterpret_cast<const __nv_bfloat16*>(p.k_cache) + (size_t)uu * kHeadDim + half * 32;
  const __nv_bfloat16* vc = reinterpret_cast<const __nv_bfloat16*>(p.v_cache) + (size_t)uu * kHeadDim + half * 32;
  uint4 q[4];                                                  // this lane's half of the query as packed bf16
  load_half(reinterpret_cast<const __nv_bfloat16*>(p.q) + (size_t)uu * kHeadDim + half * 32, q);
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;
  float o[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) o[e] = 0.f;
  float m = -INFINITY, l = 0.f;
  uint4 kr[4], vr[4], kn[4], vn[4];
  if (j0 < j1) { load_half(kc + (size_t)j0 * row_stride, kr); load_half(vc + (size_t)j0 * row_stride, vr); }
  for (int j = j0; j < j1; ++j) {
    const int jn = j + 1 < j1 ? j + 1 : j;                    // next key's rows in flight meanwhile (the last one re-read)
    load_half(kc + (size_t)jn * row_stride, kn);
    load_half(vc + (size_t)jn * row_stride, vn);
    float dt = dot_half(kr, q);
    dt += __shfl_xor_sync(0xffffffffu, dt, 1);
    const float s = dt * p.scale_log2 - slope_l2 * (float)(p.pos - j);
    const float m_new = fmaxf(m, s);
    const float corr = ex2f(m - m_new), w = ex2f(s - m_new);
    l = l * corr + w;
    m = m_new;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[8 * i] = fmaf(o[8 * i], corr, w * bf_lo_f(vr[i].x));         o[8 * i + 1] = fmaf(o[8 * i + 1], corr, w * bf_hi_f(vr[i].x));
      o[8 * i + 2] = fmaf(o[8 * i + 2], corr, w * bf_lo_f(vr[i].y)); o[8 * i + 3] = fmaf(o[8 * i + 3], corr, w * bf_hi_f(vr[i].y));
      o[8 * i + 4] = fmaf(o[8 * i + 4], corr, w * bf_lo_f(vr[i].z)); o[8 * i + 5] = fmaf(o[8 * i + 5], corr, w * bf_hi_f(vr[i].z));
      o[8 * i + 6] = fmaf(o[8 * i + 6], corr, w * bf_lo_f(vr[i].w)); o[8 * i + 7] = fmaf(o[8 * i + 7], corr, w * bf_hi_f(vr[i].w));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) { kr[i] = kn[i]; vr[i] = vn[i]; }
  }
  if (!live) return;
#pragma unroll
  for (int e = 0; e < 32; e += 2) *reinterpret_cast<float2*>(out + half * 32 + e) = make_float2(o[e], o[e + 1]);
  if (half == 0) { out[64] = m; out[65] = l; }
}

// Merges the n_chunks partial states of every pair into ONE partial state (written over the pair's first slot): a CTA
// per pair, lanes over chunks for the maximum and the weights, then lanes over the 64 dimensions with the chunks
// strided over the warps, combined through shared memory in warp order (a fixed order: bit-reproducible).
__global__ void __launch_bounds__(256) decode_attn_merge_kernel(const DecodeAttnParams p) {
  grid_dep_sync();                                           // the launches of a decode step are chained (programmatic dependent launches)
  __shared__ float s_w[kDecodeMaxRowChunks];
  __shared__ float s_red[8][68];
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* part = p.part + (size_t)u * p.n_chunks * 66;
  float mx = -INFINITY;
  for (int c = tid; c < p.n_chunks; c += 256) mx = fmaxf(mx, part[c * 66 + 64]);
  mx = warp_max(mx);
  if (lane == 0) s_red[warp][0] = mx;
  __syncthreads();
  float M = s_red[0][0];
#pragma unroll
  for (int w = 1; w < 8; ++w) M = fmaxf(M, s_red[w][0]);
  __syncthreads();
  for (int c = tid; c < p.n_chunks; c += 256) s_w[c] = ex2f(part[c * 66 + 64] - M);
  __syncthreads();
  float o0 = 0.f, o1 = 0.f, lsum = 0.f;
  for (int c = warp; c < p.n_chunks; c += 8) {                // lane = dimensions 2 lane, 2 lane + 1
    const float w = s_w[c];
    const float2 oc = *reinterpret_cast<const float2*>(part + c * 66 + 2 * lane);
    o0 = fmaf(w, oc.x, o0); o1 = fmaf(w, oc.y, o1);
    if (lane == 0) lsum = fmaf(w, part[c * 66 + 65], lsum);
  }
  s_red[warp][2 * lane] = o0; s_red[warp][2 * lane + 1] = o1;
  if (lane == 0) s_red[warp][64] = lsum;
  __syncthreads();
  if (warp == 0) {
    float a0 = 0.f, a1 = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { a0 += s_red[w][2 * lane]; a1 += s_red[w][2 * lane + 1]; ll += s_red[w][64]; }
    *reinterpret_cast<float2*>(part + 2 * lane) = make_float2(a0, a1);
    if (lane == 0) { part[64] = M; part[65] = ll; }
  }
}


// ---- pre-pass of a decode step in one launch -------------------------------------------------------------------------
// The one new row per sequence: n = RMS(x), q = qkRMS(W_q n), k~ = qkRMS(W_k n), v~ = W_v n (first display of Sec. 2.2).
// A CTA owns one head of one of the three projections (64 output columns); every CTA first normalises the B <= 16 rows
// into shared memory (they are small), then its 8 warps take 8 columns each and run the product as m16n8k16 MMAs with
// the sequences as rows, weights read straight from global memory (each weight is used once), and the head's
// normalisation is finished through shared memory.
constexpr int kPreThreads = 256;

__device__ __forceinline__ void mma_16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// a weight word that is used once: asm, so that a run of these stays a run of loads in flight
__device__ __forceinline__ uint2 ldg_stream_v2(const void* p) {
  uint2 w;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w.x), "=r"(w.y) : "l"(p));
  return w;
}
__device__ __forceinline__ unsigned pack2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const unsigned*>(&v);
}

__global__ void __launch_bounds__(kPreThreads) decode_prepass_kernel(const DecodePrepassParams p) {
  grid_dep_sync();                                           // the launches of a decode step are chained (programmatic dependent launches)
  extern __shared__ __align__(16) unsigned char dsm[];
  const int d = p.d, stride = d + 16;                          // row stride in elements: 8-byte fragment loads without conflicts
  __nv_bfloat16* n_s = reinterpret_cast<__nv_bfloat16*>(dsm);                   // [16][d + 16]
  float* ssq_s = reinterpret_cast<float*>(dsm + (size_t)16 * stride * 2);       // [8 warps][16 sequences]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool pre = (p.norm_flags & RT_NORM_PRE) != 0, qkn = (p.norm_flags & RT_NORM_QK) != 0;
  const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(p.x);
  const __nv_bfloat16* g_attn = reinterpret_cast<const __nv_bfloat16*>(p.g_attn);
  // ---- n = RMS_g(x) for the B rows (two per warp), rounded to the storage type; rows beyond B are zero ----
  for (int b = warp * 2; b < warp * 2 + 2; ++b) {
    unsigned* dst = reinterpret_cast<unsigned*>(n_s + (size_t)b * stride);
    if (b >= p.B) {
      for (int k = lane; k < d / 2; k += 32) dst[k] = 0u;
      continue;
    }
    const unsigned* xr = reinterpret_cast<const unsigned*>(x + (size_t)b * p.x_bs);
    float ss = 0.f;
    for (int k = lane; k < d / 2; k += 32) { const unsigned w = xr[k]; ss += bf_lo_f(w) * bf_lo_f(w) + bf_hi_f(w) * bf_hi_f(w); }
    ss = warp_sum(ss);
    const float rs = pre ? rsqrtf(ss / (float)d + p.eps) : 1.0f;
    for (int k = lane; k < d / 2; k += 32) {
      const unsigned w = xr[k];
      const float g0 = (pre && g_attn) ? __bfloat162float(g_attn[2 * k]) : 1.0f, g1 = (pre && g_attn) ? __bfloat162float(g_attn[2 * k + 1]) : 1.0f;
      dst[k] = pack2(bf_lo_f(w) * rs * g0, bf_hi_f(w) * rs * g1);
    }
  }
  __syncthreads();
  // ---- this warp's 8 columns of the head: sequences as MMA rows, this thread reads weight row g at k = 4c ----
  const int which = blockIdx.x / p.H, h = blockIdx.x % p.H;    // 0: q, 1: k~, 2: v~
  const __nv_bfloat16* W = reinterpret_cast<const __nv_bfloat16*>(which == 0 ? p.w_q : (which == 1 ? p.w_k : p.w_v));
  const int g = lane >> 2, c = lane & 3;
  const int col0 = h * kHeadDim + warp * 8;
  const unsigned char* wrow = reinterpret_cast<const unsigned char*>(W + (size_t)(col0 + g) * d + 4 * c);
  const unsigned char* a_lo = reinterpret_cast<const unsigned char*>(n_s + (size_t)g * stride + 4 * c);
  const unsigned char* a_hi = reinterpret_cast<const unsigned char*>(n_s + (size_t)(g + 8) * stride + 4 * c);
  float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  const int n_ks = d / 16;
  for (int ks0 = 0; ks0 < n_ks; ks0 += 16) {
    uint2 bw[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) bw[i] = ldg_stream_v2(wrow + (size_t)(ks0 + i < n_ks ? ks0 + i : ks0) * 32);   // all 16 in flight
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (ks0 + i < n_ks) {
        const size_t off = (size_t)(ks0 + i) * 32;
        const uint2 lo = *reinterpret_cast<const uint2*>(a_lo + off), hi = *reinterpret_cast<const uint2*>(a_hi + off);
        mma_16816(acc[i & 1], lo.x, hi.x, lo.y, hi.y, bw[i].x, bw[i].y);
      }
    }
  }
  float y[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) y[j] = acc[0][j] + acc[1][j];    // y0, y1: sequence g, columns col0 + 2c, + 1; y2, y3: sequence g + 8
  // ---- qkRMS over the head's 64 columns (q and k~ only), gain, storage rounding ----
  const bool norm = qkn && which < 2;
  if (norm) {
    float s_lo = y[0] * y[0] + y[1] * y[1], s_hi = y[2] * y[2] + y[3] * y[3];
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1); s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1); s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);
    if (c == 0) { ssq_s[warp * 16 + g] = s_lo; ssq_s[warp * 16 + 8 + g] = s_hi; }
  }
  __syncthreads();
  float rs_lo = 1.0f, rs_hi = 1.0f;
  if (norm) {
    float t_lo = 0.f, t_hi = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { t_lo += ssq_s[w * 16 + g]; t_hi += ssq_s[w * 16 + 8 + g]; }
    rs_lo = rsqrtf(t_lo * (1.0f / kHeadDim) + p.eps); rs_hi = rsqrtf(t_hi * (1.0f / kHeadDim) + p.eps);
  }
  const __nv_bfloat16* gain = reinterpret_cast<const __nv_bfloat16*>(which == 0 ? p.g_q : (which == 1 ? p.g_k : nullptr));
  const int col = col0 + 2 * c;
  const float ga = (norm && gain) ? __bfloat162float(gain[col]) : 1.0f, gb = (norm && gain) ? __bfloat162float(gain[col + 1]) : 1.0f;
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(which == 0 ? p.q : (which == 1 ? p.kt : p.vt));
  if (g < p.B) *reinterpret_cast<unsigned*>(out + (size_t)g * d + col) = pack2(y[0] * rs_lo * ga, y[1] * rs_lo * gb);
  if (g + 8 < p.B) *reinterpret_cast<unsigned*>(out + (size_t)(g + 8) * d + col) = pack2(y[2] * rs_hi * ga, y[3] * rs_hi * gb);
}

}  // namespace

// Chunking of a cache of `pos` positions: whole groups of 32 keys, at most kDecodeMaxChunks chunks.
int decode_attn_chunk(int pos) {
  int chunk = 64;
  while ((pos + chunk - 1) / chunk > kDecodeMaxChunks) chunk *= 2;
  return chunk;
}

cudaError_t decode_attn_launch(const DecodeAttnParams& p0, int* n_chunks, int* chunk_stride, cudaStream_t s) {
  DecodeAttnParams p = p0;
  *n_chunks = 0; *chunk_stride = 0;
  if (p.pos <= 0) return cudaSuccess;
  if (p.pos >= kDecodeRowsFrom) {
    // long cache: lane = pair, about two chunks per multiprocessor, then a parallel merge into one partial per pair
    int target = 2 * sm_count_cached();
    if (target > kDecodeMaxRowChunks) target = kDecodeMaxRowChunks;
    p.chunk = (p.pos + target - 1) / target;
    if (p.chunk < 8) p.chunk = 8;
    p.n_chunks = (p.pos + p.chunk - 1) / p.chunk;
    dim3 grid(p.n_chunks, ceil_div(2 * p.B * p.H, kRowThreads));
    { const cudaError_t el = launch_chained(decode_attn_rows_kernel, grid, dim3(kRowThreads), 0, s, true, p); if (el != cudaSuccess) return el; }
    { const cudaError_t el = launch_chained(decode_attn_merge_kernel, dim3(p.B * p.H), dim3(256), 0, s, true, p); if (el != cudaSuccess) return el; }
    *n_chunks = 1; *chunk_stride = p.n_chunks;                // the merged state sits in the pair's first slot
    return cudaGetLastError();
  }
  p.chunk = decode_attn_chunk(p.pos);
  p.n_chunks = (p.pos + p.chunk - 1) / p.chunk;
  *n_chunks = p.n_chunks; *chunk_stride = p.n_chunks;
  dim3 grid(p.n_chunks, p.B, ceil_div(p.H, kDecWarps));
  { const cudaError_t el = launch_chained(decode_attn_partial_kernel, grid, dim3(kDecWarps * 32), 0, s, true, p); if (el != cudaSuccess) return el; }
  return cudaGetLastError();
}

cudaError_t decode_prepass_launch(const DecodePrepassParams& p, cudaStream_t s) {
  const size_t smem = (size_t)16 * (p.d + 16) * 2 + 8 * 16 * 4;
  if (smem > 48 * 1024) {
    thread_local int set_for = -1;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (set_for != dev) {
      e = cudaFuncSetAttribute(decode_prepass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
      set_for = dev;
    }
  }
  { const cudaError_t el = launch_chained(decode_prepass_kernel, dim3(3 * p.H), dim3(kPreThreads), smem, s, true, p); if (el != cudaSuccess) return el; }
  return cudaGetLastError();
}

}  // namespace rt
