// Leaf recurrence kernel: the sequential part of Algorithm 1 (lines 7-12 of the loop body)
// for a run of consecutive positions, all B sequences at once.
//
// One cooperative launch = one persistent CTA per SM.  Every CTA owns a fixed slice of the
// OUTPUT rows of W_o, W_up, W_down, W_k and W_v (kept in shared memory for the whole launch
// when they fit), so a token step never re-reads weights from HBM.  A token step is five
// grid-wide phases separated by a bounded barrier:
//   A  in-launch attention: partial online-softmax states of q_t against the pairs
//      [attn_begin, t) (Algorithm 2 per 32-key batch), and qkRMS + cache write of k_{t-1}
//   B  merge partial states with the carried (m, l, o)_t, c_t = o_t / l_t, a = W_o c,
//      h = x_t + alpha a
//   C  g = GELU(W_up RMS(h))
//   D  z_t = h + alpha W_down g            (layer output, Sec. 2.2)
//   E  raw k_t = W_k RMS(z_t), v_t = W_v RMS(z_t)   (Eqs. 1-2; qkRMS of k_t happens in the next A)
// The mat-vec products split K across the 256 threads of a CTA (4 elements each per 1024-wide
// chunk) and reduce with warp shuffles, so every activation element is loaded exactly once
// per CTA and never staged.
#include "rt_kernels.h"

namespace rt {

constexpr int kLeafThreads = 256;
constexpr int kLeafWarps = kLeafThreads / 32;
constexpr int kPartStride = 68;   // partial state record: [0]=m, [1]=l, [4..67]=o

struct LeafSmemLayout {
  int max_nd, max_nf, n_rg_max;
  size_t off_red, off_ssq, off_hown, off_q, off_w, total_fixed, w_bytes;
};

static inline LeafSmemLayout leaf_smem_layout(int B, int d, int dff, int grid, int NB, size_t esize) {
  LeafSmemLayout L;
  L.max_nd = ceil_div(d, grid);
  L.max_nf = ceil_div(dff, grid);
  const int R = 32 / NB;
  int max_rows = L.max_nf > 2 * L.max_nd ? L.max_nf : 2 * L.max_nd;
  L.n_rg_max = ceil_div(max_rows, R);
  if (L.n_rg_max & 1) L.n_rg_max += 1;
  size_t o = 16;                                              // s_flag
  L.off_red = o;  o += sizeof(float) * kLeafWarps * L.n_rg_max * 32;
  L.off_ssq = o;  o += sizeof(float) * kLeafWarps * 8;
  L.off_hown = o; o += align_up(sizeof(float) * (size_t)B * L.max_nd, 16);
  L.off_q = o;    o += sizeof(float) * kLeafWarps * kHeadDim;
  o = align_up(o, 128);
  L.off_w = o;
  L.total_fixed = o;
  L.w_bytes = esize * ((size_t)L.max_nd * (3 * (size_t)d + dff) + (size_t)L.max_nf * d);
  return L;
}

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)); }

// y[row, b] = sum_k W[row, k] * act[b, k] for the CTA's rows and one group of NB sequences.
//   row_ptr(r)      -> pointer to row r (shared or global memory), r in [0, nrows)
//   load_act(b, k)  -> float4 of act[b, k..k+3] (b local to the group; zeros for padding)
//   gain            -> optional per-k gain applied to act after the sum of squares is taken
//   epi(r, b, y, ss)   ss = sum_k act[b,k]^2 (only when want_ssq)
template <typename T, int NB, typename RowPtr, typename LoadAct, typename Epi>
__device__ __forceinline__ void cta_matvec(int nrows, int K, RowPtr row_ptr, LoadAct load_act, const T* gain,
                                           bool want_ssq, Epi epi, float* red, float* ssq_red, int n_rg_max) {
  constexpr int R = 32 / NB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_rg = (nrows + R - 1) / R;
  const int n_ch = (K + 1023) / 1024;
  float ssq[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) ssq[b] = 0.f;

  for (int rg0 = 0; rg0 < n_rg; rg0 += 2) {
    float acc0[32], acc1[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) { acc0[i] = 0.f; acc1[i] = 0.f; }
    const bool two = (rg0 + 1) < n_rg;
    for (int ch = 0; ch < n_ch; ++ch) {
      const int k = ch * 1024 + 4 * tid;
      if (k < K) {
        float a[NB][4];
        float gn[4] = {1.f, 1.f, 1.f, 1.f};
        if (gain) { gn[0] = to_f(gain[k]); gn[1] = to_f(gain[k + 1]); gn[2] = to_f(gain[k + 2]); gn[3] = to_f(gain[k + 3]); }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          const float4 v = load_act(b, k);
          if (want_ssq && rg0 == 0) ssq[b] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          a[b][0] = v.x * gn[0]; a[b][1] = v.y * gn[1]; a[b][2] = v.z * gn[2]; a[b][3] = v.w * gn[3];
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int row = rg0 * R + r;
          if (row < nrows) {
            float f[4];
            reinterpret_cast<const Vec4<T>*>(row_ptr(row) + k)->to_float(f);
#pragma unroll
            for (int b = 0; b < NB; ++b)
              acc0[r * NB + b] += f[0] * a[b][0] + f[1] * a[b][1] + f[2] * a[b][2] + f[3] * a[b][3];
          }
        }
        if (two) {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int row = (rg0 + 1) * R + r;
            if (row < nrows) {
              float f[4];
              reinterpret_cast<const Vec4<T>*>(row_ptr(row) + k)->to_float(f);
#pragma unroll
              for (int b = 0; b < NB; ++b)
                acc1[r * NB + b] += f[0] * a[b][0] + f[1] * a[b][1] + f[2] * a[b][2] + f[3] * a[b][3];
            }
          }
        }
      }
    }
    warp_transpose_sum32(acc0, lane);
    red[(warp * n_rg_max + rg0) * 32 + lane] = acc0[0];
    if (two) {
      warp_transpose_sum32(acc1, lane);
      red[(warp * n_rg_max + rg0 + 1) * 32 + lane] = acc1[0];
    }
  }
  if (want_ssq) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const float s = warp_sum(ssq[b]);
      if (lane == 0) ssq_red[warp * 8 + b] = s;
    }
  }
  __syncthreads();
  for (int idx = tid; idx < n_rg * 32; idx += kLeafThreads) {
    const int rg = idx >> 5, i = idx & 31;
    const int r = i / NB, b = i % NB;
    const int row = rg * R + r;
    if (row < nrows) {
      float v = 0.f, ss = 0.f;
#pragma unroll
      for (int w = 0; w < kLeafWarps; ++w) v += red[(w * n_rg_max + rg) * 32 + i];
      if (want_ssq) {
#pragma unroll
        for (int w = 0; w < kLeafWarps; ++w) ss += ssq_red[w * 8 + b];
      }
      epi(row, b, v, ss);
    }
  }
  __syncthreads();
}

template <typename T, int NB>
__global__ void __launch_bounds__(kLeafThreads, 1) leaf_kernel(const LeafParams p, const LeafSmemLayout L) {
  extern __shared__ __align__(128) unsigned char smem[];
  int* s_flag = reinterpret_cast<int*>(smem);
  float* red = reinterpret_cast<float*>(smem + L.off_red);
  float* ssq_red = reinterpret_cast<float*>(smem + L.off_ssq);
  float* hown = reinterpret_cast<float*>(smem + L.off_hown);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int B = p.B, d = p.d, H = p.H, dff = p.dff;
  // an earlier launch of this call gave up: its barrier count is short, do not wait on it
  if (*reinterpret_cast<volatile unsigned*>(&p.sync->abort_flag)) return;
  const int d_lo = (int)((long long)d * cta / G), d_hi = (int)((long long)d * (cta + 1) / G);
  const int f_lo = (int)((long long)dff * cta / G), f_hi = (int)((long long)dff * (cta + 1) / G);
  const int nd = d_hi - d_lo, nf = f_hi - f_lo;
  const bool pre = (p.norm_flags & RT_NORM_PRE) != 0;
  const bool qkn = (p.norm_flags & RT_NORM_QK) != 0;
  const bool kv_norm = pre && !(p.norm_flags & RT_NORM_SKIP_Z);

  const T* Wo = reinterpret_cast<const T*>(p.w_o) + (size_t)d_lo * d;
  const T* Wup = reinterpret_cast<const T*>(p.w_up) + (size_t)f_lo * d;
  const T* Wdn = reinterpret_cast<const T*>(p.w_down) + (size_t)d_lo * dff;
  const T* Wk = reinterpret_cast<const T*>(p.w_k) + (size_t)d_lo * d;
  const T* Wv = reinterpret_cast<const T*>(p.w_v) + (size_t)d_lo * d;
  if (p.weights_in_smem) {
    T* sw = reinterpret_cast<T*>(smem + L.off_w);
    T* s_o = sw;
    T* s_up = s_o + (size_t)L.max_nd * d;
    T* s_dn = s_up + (size_t)L.max_nf * d;
    T* s_k = s_dn + (size_t)L.max_nd * dff;
    T* s_v = s_k + (size_t)L.max_nd * d;
    auto copy_rows = [&](T* dst, const T* src, size_t n_elems) {
      const uint4* s4 = reinterpret_cast<const uint4*>(src);
      uint4* d4 = reinterpret_cast<uint4*>(dst);
      const size_t n4 = n_elems * sizeof(T) / 16;
      for (size_t i = tid; i < n4; i += kLeafThreads) d4[i] = s4[i];
    };
    copy_rows(s_o, Wo, (size_t)nd * d);
    copy_rows(s_up, Wup, (size_t)nf * d);
    copy_rows(s_dn, Wdn, (size_t)nd * dff);
    copy_rows(s_k, Wk, (size_t)nd * d);
    copy_rows(s_v, Wv, (size_t)nd * d);
    Wo = s_o; Wup = s_up; Wdn = s_dn; Wk = s_k; Wv = s_v;
    __syncthreads();
  }

  const T* g_mlp = reinterpret_cast<const T*>(p.g_mlp);
  const T* g_kv = reinterpret_cast<const T*>(p.g_kv);
  const T* g_k = reinterpret_cast<const T*>(p.g_k);
  const T* xq = reinterpret_cast<const T*>(p.q);
  const T* x = reinterpret_cast<const T*>(p.x);
  T* z = reinterpret_cast<T*>(p.z);
  T* kc = reinterpret_cast<T*>(p.k_cache);
  T* vc = reinterpret_cast<T*>(p.v_cache);
  const float inv_d = 1.0f / (float)d;
  unsigned bar_target = p.bar_base;
  const int n_bg = (B + NB - 1) / NB;

  // phase timing by one thread of CTA 0 (two timer reads per phase)
  const bool timing = p.timers && (cta == 0 && tid == 0);
  unsigned long long t_prev = timing ? globaltimer_ns() : 0ull, acc_ns[10];
#pragma unroll
  for (int i = 0; i < 10; ++i) acc_ns[i] = 0ull;
#define LEAF_PHASE_END(i)                                                   \
  {                                                                         \
    unsigned long long t_a = timing ? globaltimer_ns() : 0ull;              \
    const bool ok_ = grid_barrier(p.sync, bar_target, G, s_flag);           \
    if (timing) {                                                           \
      const unsigned long long t_b = globaltimer_ns();                      \
      acc_ns[2 * (i)] += t_a - t_prev;                                      \
      acc_ns[2 * (i) + 1] += t_b - t_a;                                     \
      t_prev = t_b;                                                         \
    }                                                                       \
    if (!ok_) return;                                                       \
  }

  for (int t = p.t0; t < p.t1; ++t) {
    const int row = t - p.row_off;
    // ---------------- phase A: partial attention over the pairs [attn_begin, t) ----------------
    const int nkeys = t - p.attn_begin;
    int nch = 0, per = 0;
    if (nkeys > 0) {
      nch = (nkeys + 31) / 32;
      if (nch > p.max_chunks) nch = p.max_chunks;
      per = ((nkeys + nch - 1) / nch + 31) & ~31;
      nch = (nkeys + per - 1) / per;
      const int units = B * H * nch;
      for (int u = cta + G * warp; u < units; u += G * kLeafWarps) {
        const int c = u % nch, bh = u / nch, b = bh / H, h = bh % H;
        const int j0 = p.attn_begin + c * per;
        const int j1 = (j0 + per < t) ? j0 + per : t;
        const T* qrow = xq + ((size_t)row * B + b) * d + h * kHeadDim;
        const float q0 = to_f(qrow[2 * lane]), q1 = to_f(qrow[2 * lane + 1]);      // this lane's two dimensions
        const float slope_l2 = p.alibi ? p.alibi[h] * kLog2e : 0.f;                 // ALiBi distances, log2 units
        // The pair revealed by the previous step of this launch is still un-normalised in ex_k: the warp
        // applies qkRMS (Eq. 1), writes the cache row and keeps the rounded values for its own product.
        const bool fresh = (t - 1 >= p.t0) && (t - 1 >= j0) && (t - 1 < j1);
        float kn0 = 0.f, kn1 = 0.f;
        if (fresh) {
          const float2 r2 = __ldcg(reinterpret_cast<const float2*>(p.ex_k + (size_t)b * d + h * kHeadDim + 2 * lane));
          const float ss = warp_sum(r2.x * r2.x + r2.y * r2.y);
          const float rs = qkn ? rsqrtf(ss * (1.0f / kHeadDim) + p.eps) : 1.0f;
          const float g0 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane) : 1.0f;
          const float g1 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane + 1) : 1.0f;
          T* kdst = kc + ((size_t)(t - 1) * B + b) * d + h * kHeadDim + 2 * lane;
          const T ka = from_f<T>(r2.x * rs * g0), kb = from_f<T>(r2.y * rs * g1);
          kdst[0] = ka; kdst[1] = kb;
          kn0 = to_f(ka); kn1 = to_f(kb);
        }
        float m_run = -INFINITY, l_run = 0.f, o0 = 0.f, o1 = 0.f;
        for (int jb = j0; jb < j1; jb += 32) {
          const int cnt = (j1 - jb < 32) ? (j1 - jb) : 32;
          // K: one coalesced row load per key (lanes over the head's dimensions), all 32 in flight, then a
          // transposed reduction leaves the score of key jb + lane in this lane
          float prod[32];
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const int j = jb + (jj < cnt ? jj : 0);
            float2 k2 = ldcg_T2(kc + ((size_t)j * B + b) * d + h * kHeadDim + 2 * lane);
            if (fresh && j == t - 1) k2 = make_float2(kn0, kn1);
            prod[jj] = q0 * k2.x + q1 * k2.y;
          }
          // V rows of the batch, requested before the scores are needed
          float2 vv[32];
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const int j = jb + (jj < cnt ? jj : 0);
            vv[jj] = ldcg_T2(vc + ((size_t)j * B + b) * d + h * kHeadDim + 2 * lane);
          }
          warp_transpose_sum32(prod, lane);
          const bool valid = lane < cnt;
          const float s2 = valid ? prod[0] * p.scale_log2 - slope_l2 * (float)(t - (jb + lane)) : -INFINITY;
          const float m_new = fmaxf(m_run, warp_max(s2));
          const float pj = valid ? exp2f(s2 - m_new) : 0.f;
          const float corr = exp2f(m_run - m_new);
          l_run = l_run * corr + warp_sum(pj);
          o0 *= corr; o1 *= corr;
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const float pw = __shfl_sync(0xffffffffu, pj, jj);       // 0 for the keys beyond cnt
            o0 += pw * vv[jj].x; o1 += pw * vv[jj].y;
          }
          m_run = m_new;
        }
        float* part = p.ex_part + ((size_t)bh * p.max_chunks + c) * kPartStride;
        if (lane == 0) { part[0] = m_run; part[1] = l_run; }
        *reinterpret_cast<float2*>(part + 4 + 2 * lane) = make_float2(o0, o1);
      }
    }
    LEAF_PHASE_END(0);

    // ---------------- phase B: c_t = merged state / l, a = W_o c, h = x_t + alpha a ----------------
    for (int bg = 0; bg < n_bg; ++bg) {
      auto load_c = [&](int bl, int k) -> float4 {
        const int b = bg * NB + bl;
        if (b >= B) return make_float4(0.f, 0.f, 0.f, 0.f);
        const int h = k / kHeadDim, e = k % kHeadDim;
        const size_t sidx = ((size_t)row * B + b);
        float m = p.st_m[sidx * H + h], l = p.st_l[sidx * H + h];
        float4 o = *reinterpret_cast<const float4*>(p.st_o + sidx * d + k);
        const float* part = p.ex_part + ((size_t)(b * H + h) * p.max_chunks) * kPartStride;
        for (int c = 0; c < nch; ++c, part += kPartStride) {
          const float pm = ldcg_f(part), pl = ldcg_f(part + 1);
          const float4 po = ldcg_f4(part + 4 + e);
          const float mn = fmaxf(m, pm);
          const float fa = exp2f(m - mn), fb = exp2f(pm - mn);
          l = l * fa + pl * fb;
          o.x = o.x * fa + po.x * fb; o.y = o.y * fa + po.y * fb;
          o.z = o.z * fa + po.z * fb; o.w = o.w * fa + po.w * fb;
          m = mn;
        }
        const float il = 1.0f / l;
        return make_float4(o.x * il, o.y * il, o.z * il, o.w * il);
      };
      auto epi = [&](int r, int bl, float v, float) {
        const int b = bg * NB + bl;
        if (b >= B) return;
        const int grow = d_lo + r;
        const float xv = to_f(x[(size_t)b * p.x_bs + (size_t)row * p.x_ts + grow]);
        const float hv = xv + p.alpha * v;
        p.ex_h[(size_t)b * d + grow] = hv;
        hown[b * L.max_nd + r] = hv;
      };
      cta_matvec<T, NB>(nd, d, [&](int r) { return Wo + (size_t)r * d; }, load_c, (const T*)nullptr, false, epi,
                        red, ssq_red, L.n_rg_max);
    }
    LEAF_PHASE_END(1);

    // ---------------- phase C: g = GELU(W_up RMS(h)) ----------------
    for (int bg = 0; bg < n_bg; ++bg) {
      auto load_h = [&](int bl, int k) -> float4 {
        const int b = bg * NB + bl;
        if (b >= B) return make_float4(0.f, 0.f, 0.f, 0.f);
        return ldcg_f4(p.ex_h + (size_t)b * d + k);
      };
      auto epi = [&](int r, int bl, float v, float ss) {
        const int b = bg * NB + bl;
        if (b >= B) return;
        const float rs = pre ? rsqrtf(ss * inv_d + p.eps) : 1.0f;
        p.ex_g[(size_t)b * dff + f_lo + r] = gelu_erf(v * rs);
      };
      cta_matvec<T, NB>(nf, d, [&](int r) { return Wup + (size_t)r * d; }, load_h, pre ? g_mlp : (const T*)nullptr,
                        pre, epi, red, ssq_red, L.n_rg_max);
    }
    LEAF_PHASE_END(2);

    // ---------------- phase D: z_t = h + alpha W_down g ----------------
    for (int bg = 0; bg < n_bg; ++bg) {
      auto load_g = [&](int bl, int k) -> float4 {
        const int b = bg * NB + bl;
        if (b >= B) return make_float4(0.f, 0.f, 0.f, 0.f);
        return ldcg_f4(p.ex_g + (size_t)b * dff + k);
      };
      auto epi = [&](int r, int bl, float v, float) {
        const int b = bg * NB + bl;
        if (b >= B) return;
        const int grow = d_lo + r;
        const float zv = hown[b * L.max_nd + r] + p.alpha * v;
        p.ex_z[(size_t)b * d + grow] = zv;
        z[(size_t)b * p.z_bs + (size_t)row * p.z_ts + grow] = from_f<T>(zv);
      };
      cta_matvec<T, NB>(nd, dff, [&](int r) { return Wdn + (size_t)r * dff; }, load_g, (const T*)nullptr, false, epi,
                        red, ssq_red, L.n_rg_max);
    }
    LEAF_PHASE_END(3);

    // ---------------- phase E: raw k_t = W_k RMS(z_t), v_t = W_v RMS(z_t) ----------------
    for (int bg = 0; bg < n_bg; ++bg) {
      auto load_z = [&](int bl, int k) -> float4 {
        const int b = bg * NB + bl;
        if (b >= B) return make_float4(0.f, 0.f, 0.f, 0.f);
        return ldcg_f4(p.ex_z + (size_t)b * d + k);
      };
      auto epi = [&](int r, int bl, float v, float ss) {
        const int b = bg * NB + bl;
        if (b >= B) return;
        const float rs = kv_norm ? rsqrtf(ss * inv_d + p.eps) : 1.0f;
        if (r < nd) p.ex_k[(size_t)b * d + d_lo + r] = v * rs;
        else vc[((size_t)t * B + b) * d + d_lo + (r - nd)] = from_f<T>(v * rs);
      };
      cta_matvec<T, NB>(2 * nd, d,
                        [&](int r) { return r < nd ? Wk + (size_t)r * d : Wv + (size_t)(r - nd) * d; }, load_z,
                        kv_norm ? g_kv : (const T*)nullptr, kv_norm, epi, red, ssq_red, L.n_rg_max);
    }
    LEAF_PHASE_END(4);
  }

  if (timing) {
#pragma unroll
    for (int i = 0; i < 10; ++i) atomicAdd(&p.sync->phase_ns[i], acc_ns[i]);
  }
#undef LEAF_PHASE_END

  // ---------------- qkRMS and cache write of the last key of this launch ----------------
  if (p.t1 > p.t0) {
    const int t = p.t1 - 1;
    for (int u = cta + G * warp; u < B * H; u += G * kLeafWarps) {
      const int b = u / H, h = u % H;
      const float2 r2 = ldcg_T2(p.ex_k + (size_t)b * d + h * kHeadDim + 2 * lane);
      const float ss = warp_sum(r2.x * r2.x + r2.y * r2.y);
      const float rs = qkn ? rsqrtf(ss * (1.0f / kHeadDim) + p.eps) : 1.0f;
      const float g0 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane) : 1.0f;
      const float g1 = qkn ? gain_at(g_k, h * kHeadDim + 2 * lane + 1) : 1.0f;
      T* kdst = kc + ((size_t)t * B + b) * d + h * kHeadDim + 2 * lane;
      kdst[0] = from_f<T>(r2.x * rs * g0);
      kdst[1] = from_f<T>(r2.y * rs * g1);
    }
  }
}

// Self-test of the bounded wait: the barrier below expects one more arrival than there are CTAs,
// so it can only end through the time limit.
__global__ void wait_expiry_selftest_kernel(SyncArea* sync) {
  __shared__ int s_flag;
  unsigned target = 0;
  grid_barrier(sync, target, gridDim.x + 1, &s_flag);
}

cudaError_t wait_expiry_selftest_launch(SyncArea* sync, cudaStream_t s) {
  void* args[] = {(void*)&sync};
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(&wait_expiry_selftest_kernel), dim3(2), dim3(32), args, 0, s);
}

// ------------------------------------------------------------------------------------ host

static inline int pick_nb(int B) { return B > 4 ? 8 : (B > 2 ? 4 : (B > 1 ? 2 : 1)); }

template <typename T>
static const void* leaf_fn(int NB) {
  switch (NB) {
    case 1: return reinterpret_cast<const void*>(&leaf_kernel<T, 1>);
    case 2: return reinterpret_cast<const void*>(&leaf_kernel<T, 2>);
    case 4: return reinterpret_cast<const void*>(&leaf_kernel<T, 4>);
    default: return reinterpret_cast<const void*>(&leaf_kernel<T, 8>);
  }
}

cudaError_t leaf_plan(int dtype, int B, int d, int dff, LeafLaunch* out) {
  int dev = 0, sms = 0, max_smem = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
  const size_t esize = dtype == RT_BF16 ? 2 : 4;
  const int NB = pick_nb(B);
  const LeafSmemLayout L = leaf_smem_layout(B, d, dff, sms, NB, esize);
  out->grid = sms;
  out->block = kLeafThreads;
  out->weights_in_smem = (L.total_fixed + L.w_bytes <= (size_t)max_smem) ? 1 : 0;
  out->smem = L.total_fixed + (out->weights_in_smem ? L.w_bytes : 0);
  if (out->smem > (size_t)max_smem) return cudaErrorInvalidConfiguration;
  return cudaSuccess;
}

cudaError_t leaf_launch(int dtype, const LeafParams& p_in, const LeafLaunch& l, cudaStream_t s) {
  LeafParams p = p_in;
  p.weights_in_smem = l.weights_in_smem;
  const size_t esize = dtype == RT_BF16 ? 2 : 4;
  const int NB = pick_nb(p.B);
  LeafSmemLayout L = leaf_smem_layout(p.B, p.d, p.dff, l.grid, NB, esize);
  const void* fn = dtype == RT_BF16 ? leaf_fn<__nv_bfloat16>(NB) : leaf_fn<float>(NB);
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.smem);
  if (e != cudaSuccess) return e;
  void* args[] = {(void*)&p, (void*)&L};
  return cudaLaunchCooperativeKernel(fn, dim3(l.grid), dim3(l.block), args, l.smem, s);
}

}  // namespace rt
