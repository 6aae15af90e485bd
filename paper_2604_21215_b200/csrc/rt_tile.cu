// Cross-block tile: Algorithm 2 (UpdateTile) applied to queries [q0,q1) against the revealed
// pairs [k0,k1), for every sequence and head, with the running stats (m, l, o) carried in
// fp32 between tiles.  This file holds the SIMT version (fp32 mode, and any shape the
// tensor-core version does not take).  m is kept in log2 units: p = 2^(s*log2e*<q,k> - m).
// With ALiBi distances the logit of query i on pair j also gets -slope_h (i - j) (times log2e).
#include "rt_kernels.h"

namespace rt {

constexpr int kTQ = 16;    // query rows per CTA
constexpr int kTK = 32;    // keys per shared-memory chunk

template <typename T>
__global__ void __launch_bounds__(128) tile_simt_kernel(const TileParams p) {
  __shared__ float Qs[kTQ][kHeadDim];
  __shared__ float Ks[kTK][kHeadDim + 1];
  __shared__ float Vs[kTK][kHeadDim];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  const int shift = (int)blockIdx.z * p.batch_stride;                   // copy z of the tile (one level in one launch)
  const int q0 = p.q0 + shift, k0 = p.k0 + shift;
  int q1 = p.q1 + shift, k1 = p.k1 + shift;
  if (p.q_limit > 0 && q1 > p.q_limit) q1 = p.q_limit;
  if (p.q_limit > 0 && k1 > p.q_limit) k1 = p.q_limit;         // (a causal block's keys end where its queries do)
  const int qb = q0 + blockIdx.x * kTQ;
  if (qb >= q1) return;
  const T* Q = reinterpret_cast<const T*>(p.q);
  const T* Kc = reinterpret_cast<const T*>(p.k_cache);
  const T* Vc = reinterpret_cast<const T*>(p.v_cache);
  const size_t col0 = (size_t)b * p.d + h * kHeadDim;
  const size_t rstride = (size_t)p.B * p.d;
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;

  for (int i = tid; i < kTQ * kHeadDim; i += 128) {
    const int r = i / kHeadDim, e = i % kHeadDim;
    Qs[r][e] = (qb + r < q1) ? to_f(Q[(size_t)(qb + r) * rstride + col0 + e]) : 0.f;
  }
  // each warp owns 4 query rows; lane holds dims lane and lane+32 of o
  float m[4], l[4], oa[4], ob[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int qi = qb + warp * 4 + i;
    if (qi < q1) {
      const size_t sidx = (size_t)qi * p.B + b;
      m[i] = p.st_m[sidx * p.H + h];
      l[i] = p.st_l[sidx * p.H + h];
      oa[i] = p.st_o[sidx * p.d + h * kHeadDim + lane];
      ob[i] = p.st_o[sidx * p.d + h * kHeadDim + lane + 32];
    } else { m[i] = 0.f; l[i] = 0.f; oa[i] = 0.f; ob[i] = 0.f; }
  }
  for (int kb = k0; kb < k1; kb += kTK) {
    __syncthreads();
    for (int i = tid; i < kTK * kHeadDim; i += 128) {
      const int r = i / kHeadDim, e = i % kHeadDim;
      const bool ok = kb + r < k1;
      Ks[r][e] = ok ? to_f(Kc[(size_t)(kb + r) * rstride + col0 + e]) : 0.f;
      Vs[r][e] = ok ? to_f(Vc[(size_t)(kb + r) * rstride + col0 + e]) : 0.f;
    }
    __syncthreads();
    const bool in_range = kb + lane < k1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int qr = warp * 4 + i;
      const bool valid = in_range && (!p.causal || kb + lane < qb + qr);   // causal: only earlier positions
      if (p.causal && kb >= qb + qr) continue;                            // whole chunk masked for this row (warp-uniform)
      float s = 0.f;
#pragma unroll 16
      for (int e = 0; e < kHeadDim; ++e) s += Qs[qr][e] * Ks[lane][e];
      const float s2 = valid ? s * p.scale_log2 - slope_l2 * (float)(qb + qr - (kb + lane)) : -INFINITY;
      const float m_new = fmaxf(m[i], warp_max(s2));
      const float pj = valid ? exp2f(s2 - m_new) : 0.f;
      const float corr = exp2f(m[i] - m_new);
      l[i] = l[i] * corr + warp_sum(pj);
      float a = oa[i] * corr, c = ob[i] * corr;
#pragma unroll 8
      for (int jj = 0; jj < kTK; ++jj) {
        const float pw = __shfl_sync(0xffffffffu, pj, jj);
        a += pw * Vs[jj][lane];
        c += pw * Vs[jj][lane + 32];
      }
      oa[i] = a; ob[i] = c; m[i] = m_new;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int qi = qb + warp * 4 + i;
    if (qi < q1) {
      const size_t sidx = (size_t)qi * p.B + b;
      if (lane == 0) { p.st_m[sidx * p.H + h] = m[i]; p.st_l[sidx * p.H + h] = l[i]; }
      p.st_o[sidx * p.d + h * kHeadDim + lane] = oa[i];
      p.st_o[sidx * p.d + h * kHeadDim + lane + 32] = ob[i];
    }
  }
}

cudaError_t tile_simt_launch(int dtype, const TileParams& p, cudaStream_t s) {
  const int nq = p.q1 - p.q0;
  if (nq <= 0 || p.k1 <= p.k0) return cudaSuccess;
  dim3 grid(ceil_div(nq, kTQ), p.B * p.H, p.batch > 1 ? p.batch : 1);
  if (dtype == RT_BF16) tile_simt_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(p);
  else tile_simt_kernel<float><<<grid, 128, 0, s>>>(p);
  return cudaGetLastError();
}

// ---- one query row per (sequence, head) against a short run of pairs -----------------------------------
// Used by the wide-batch token step: position t attends to the pairs of its own leaf revealed so far,
// [k0, k1) with k1 = t.  One warp per (sequence, head): each K and V row is one coalesced load (lanes over
// the head's dimensions), the 32 per-lane partial products become per-key scores by a transposed reduction.
template <typename T, int G>
__global__ void __launch_bounds__(256) row_attn_kernel(const TileParams p) {
  // G: groups of 8 keys fetched per batch of 32 (the launcher picks the smallest that covers k1 - k0 when that is at most 32)
  grid_dep_sync();
  const int lane = threadIdx.x & 31;
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (u >= p.B * p.H) return;
  const int b = u / p.H, h = u % p.H;
  const int t = p.q0;
  const T* Kc = reinterpret_cast<const T*>(p.k_cache);
  const T* Vc = reinterpret_cast<const T*>(p.v_cache);
  const size_t col = (size_t)b * p.d + h * kHeadDim + 2 * lane;
  const size_t rstride = (size_t)p.B * p.d;
  const T* qrow = reinterpret_cast<const T*>(p.q) + (size_t)t * rstride + col;
  const float q0 = to_f(qrow[0]), q1 = to_f(qrow[1]);
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;
  const size_t sidx = (size_t)t * p.B + b;
  float m_run = p.st_m[sidx * p.H + h], l_run = p.st_l[sidx * p.H + h];
  float2 o = *reinterpret_cast<const float2*>(p.st_o + sidx * p.d + h * kHeadDim + 2 * lane);
  for (int jb = p.k0; jb < p.k1; jb += 32) {
    const int cnt = (p.k1 - jb < 32) ? (p.k1 - jb) : 32;
    float prod[32];
    float2 vv[32];
#pragma unroll
    for (int jj = 0; jj < 32; ++jj) {
      if (jj < 8 * G) {
        const int j = jb + (jj < cnt ? jj : 0);
        const float2 k2 = ldcg_T2(Kc + (size_t)j * rstride + col);
        vv[jj] = ldcg_T2(Vc + (size_t)j * rstride + col);
        prod[jj] = q0 * k2.x + q1 * k2.y;
      } else {
        prod[jj] = 0.f;
      }
    }
    warp_transpose_sum32(prod, lane);
    const bool valid = lane < cnt;
    const float s2 = valid ? prod[0] * p.scale_log2 - slope_l2 * (float)(t - (jb + lane)) : -INFINITY;
    const float m_new = fmaxf(m_run, warp_max(s2));
    const float pj = valid ? exp2f(s2 - m_new) : 0.f;
    const float corr = exp2f(m_run - m_new);
    l_run = l_run * corr + warp_sum(pj);
    o.x *= corr; o.y *= corr;
#pragma unroll
    for (int jj = 0; jj < 8 * G; ++jj) {
      const float pw = __shfl_sync(0xffffffffu, pj, jj);
      o.x += pw * vv[jj].x; o.y += pw * vv[jj].y;
    }
    m_run = m_new;
  }
  if (lane == 0) { p.st_m[sidx * p.H + h] = m_run; p.st_l[sidx * p.H + h] = l_run; }
  *reinterpret_cast<float2*>(p.st_o + sidx * p.d + h * kHeadDim + 2 * lane) = o;
  if (p.c_out) {                                               // the row is complete: c = o / l for the output projection
    const float il = 1.0f / l_run;
    T* c = reinterpret_cast<T*>(p.c_out) + col;
    c[0] = from_f<T>(o.x * il); c[1] = from_f<T>(o.y * il);
  }
}

cudaError_t row_attn_launch(int dtype, const TileParams& p, cudaStream_t s) {
  if (p.k1 <= p.k0 && !p.c_out) return cudaSuccess;
  const int blocks = ceil_div(p.B * p.H, 8);
  const int nk = p.k1 - p.k0;
  const int groups = nk > 32 ? 4 : (nk > 24 ? 4 : (nk > 16 ? 3 : (nk > 8 ? 2 : 1)));
  auto go = [&](auto kern) { return launch_chained(kern, dim3(blocks), dim3(256), 0, s, p.chained != 0, p); };
  if (dtype == RT_BF16) {
    switch (groups) {
      case 1: return go(row_attn_kernel<__nv_bfloat16, 1>);
      case 2: return go(row_attn_kernel<__nv_bfloat16, 2>);
      case 3: return go(row_attn_kernel<__nv_bfloat16, 3>);
      default: return go(row_attn_kernel<__nv_bfloat16, 4>);
    }
  }
  switch (groups) {
    case 1: return go(row_attn_kernel<float, 1>);
    case 2: return go(row_attn_kernel<float, 2>);
    case 3: return go(row_attn_kernel<float, 3>);
    default: return go(row_attn_kernel<float, 4>);
  }
}

// ---- small tiles: at most 16 pairs against a short run of queries ---------------------------------------
// Algorithm 2 for the lowest levels of a short-leaf schedule (wide batches: leaves of 16).  One warp per (sequence,
// head) and kSmallTileQueries queries: the K and V rows of the tile are fetched once (one coalesced load per row, lanes
// over the head's dimensions) and stay in registers, and the warp's query rows, output rows and statistics are all
// requested before the first product; every query then costs one transposed reduction for its scores and one pass over
// the values.  G = groups of 8 pairs (1 or 2).
constexpr int kSmallTileQueries = 4;      // queries per warp
template <typename T, int G>
__global__ void __launch_bounds__(128) tile_rows_kernel(const TileParams p) {
  grid_dep_sync();
  const int lane = threadIdx.x & 31;
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (u >= p.B * p.H) return;
  const int b = u / p.H, h = u % p.H;
  const int qa = p.q0 + (int)blockIdx.y * kSmallTileQueries;
  const int cnt = p.k1 - p.k0;
  const T* Kc = reinterpret_cast<const T*>(p.k_cache);
  const T* Vc = reinterpret_cast<const T*>(p.v_cache);
  const size_t col = (size_t)b * p.d + h * kHeadDim + 2 * lane;
  const size_t rstride = (size_t)p.B * p.d;
  const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;
  float2 qq[kSmallTileQueries], oo[kSmallTileQueries];
  float mm[kSmallTileQueries], ll[kSmallTileQueries];
#pragma unroll
  for (int i = 0; i < kSmallTileQueries; ++i) {
    const int t = qa + i < p.q1 ? qa + i : p.q1 - 1;              // (rows beyond the tile repeat its last query and are not stored)
    const size_t sidx = (size_t)t * p.B + b;
    qq[i] = ldcg_T2(reinterpret_cast<const T*>(p.q) + (size_t)t * rstride + col);
    oo[i] = __ldcg(reinterpret_cast<const float2*>(p.st_o + sidx * p.d + h * kHeadDim + 2 * lane));
    mm[i] = __ldcg(p.st_m + sidx * p.H + h);
    ll[i] = __ldcg(p.st_l + sidx * p.H + h);
  }
  float2 kk[8 * G], vv[8 * G];
#pragma unroll
  for (int jj = 0; jj < 8 * G; ++jj) {
    const int j = p.k0 + (jj < cnt ? jj : 0);
    kk[jj] = ldcg_T2(Kc + (size_t)j * rstride + col);
    vv[jj] = ldcg_T2(Vc + (size_t)j * rstride + col);
  }
  const bool valid = lane < cnt;
#pragma unroll
  for (int i = 0; i < kSmallTileQueries; ++i) {
    const int t = qa + i;
    float prod[32];
#pragma unroll
    for (int jj = 0; jj < 32; ++jj) prod[jj] = jj < 8 * G ? qq[i].x * kk[jj].x + qq[i].y * kk[jj].y : 0.f;
    warp_transpose_sum32(prod, lane);
    const float s2 = valid ? prod[0] * p.scale_log2 - slope_l2 * (float)(t - (p.k0 + lane)) : -INFINITY;
    const float m_new = fmaxf(mm[i], warp_max(s2));
    const float pj = valid ? exp2f(s2 - m_new) : 0.f;
    const float corr = exp2f(mm[i] - m_new);
    const float l_new = ll[i] * corr + warp_sum(pj);
    float2 o = make_float2(oo[i].x * corr, oo[i].y * corr);
#pragma unroll
    for (int jj = 0; jj < 8 * G; ++jj) {
      const float pw = __shfl_sync(0xffffffffu, pj, jj);
      o.x += pw * vv[jj].x; o.y += pw * vv[jj].y;
    }
    if (t < p.q1) {
      const size_t sidx = (size_t)t * p.B + b;
      if (lane == 0) { p.st_m[sidx * p.H + h] = m_new; p.st_l[sidx * p.H + h] = l_new; }
      *reinterpret_cast<float2*>(p.st_o + sidx * p.d + h * kHeadDim + 2 * lane) = o;
    }
  }
}

cudaError_t tile_rows_launch(int dtype, const TileParams& p, cudaStream_t s) {
  const int nk = p.k1 - p.k0, nq = p.q1 - p.q0;
  dim3 grid(ceil_div(p.B * p.H, 4), ceil_div(nq, kSmallTileQueries));
  auto go = [&](auto kern) { return launch_chained(kern, grid, dim3(128), 0, s, p.chained != 0, p); };
  if (dtype == RT_BF16) return nk > 8 ? go(tile_rows_kernel<__nv_bfloat16, 2>) : go(tile_rows_kernel<__nv_bfloat16, 1>);
  return nk > 8 ? go(tile_rows_kernel<float, 2>) : go(tile_rows_kernel<float, 1>);
}

cudaError_t tile_launch(int dtype, const TileParams& p, cudaStream_t s) {
  // at most 16 pairs, a plain tile (no causal mask, one copy): the small-tile kernel (measured on B = 512, H = 16: 16 pairs
  // x 16 queries 78 us against 127 us; with 32 pairs the registers it needs leave too few warps per SM: 260 against 254 us)
  if (p.k1 - p.k0 <= 16 && p.k1 > p.k0 && p.q1 > p.q0 && !p.causal && p.batch <= 1 && p.q_limit == 0)
    return tile_rows_launch(dtype, p, s);
  // Whole 64-key blocks only on the tensor-core path: a partial block would bring cache rows that
  // are not revealed yet (arbitrary bits) into the P.V product.
  if (dtype == RT_BF16 && (p.k1 - p.k0) % 64 == 0 && p.d % kHeadDim == 0)
    return tile_tc_launch(p, p.rows_q, p.rows_kv, p.sync, s);
  return tile_simt_launch(dtype, p, s);
}

}  // namespace rt
