// C ABI of the library (see include/rt.h): argument checks, workspace layout, and the
// schedule of Algorithm 1 at leaf granularity -- solve a leaf, then let the next query block
// attend to the block of pairs that just became complete.
#include <math.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "rt_kernels.h"

using namespace rt;

namespace {

constexpr int kMaxChunks = 32;
constexpr int kSmallBatchMax = 64;      // above this the per-token chain runs as dense products (tiled prefill only)
constexpr int kAutoLeaf = 64;

struct WsLayout {
  size_t sync, q, kt, vt, n, st_o, st_m, st_l, ex_h, ex_g, ex_z, ex_k, ex_part, dec_part, ll, ll_bytes, hid0, hid1,
      blk_h, blk_u, blk_c, blk_g, total;
};

size_t esize_of(int dtype) { return dtype == RT_BF16 ? 2 : 4; }

bool config_ok(const rt_config* c) {
  if (!c) return false;
  if (c->d_model <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->d_ff <= 0) return false;
  if ((long long)c->n_heads * c->head_dim != c->d_model) return false;
  if (c->dtype != RT_F32 && c->dtype != RT_BF16) return false;
  if (c->sched != RT_SCHED_TILED && c->sched != RT_SCHED_NAIVE) return false;
  if (c->leaf != 0 && (c->leaf < 16 || c->leaf > 256 || (c->leaf & (c->leaf - 1)))) return false;
  if (!(c->rms_eps >= 0.f) || !isfinite(c->softmax_scale) || !isfinite(c->residual_scale)) return false;
  if (c->norm_flags & ~(RT_NORM_PRE | RT_NORM_QK | RT_NORM_SKIP_Z)) return false;
  if (c->recur_block < 0) return false;
  if (c->flags & ~RT_FLAG_BACKWARD_STEP_LAUNCHES) return false;
  return true;
}

rt_status config_supported(const rt_config* c, int B, bool wide_ok = false) {
  if (c->head_dim != kHeadDim) return RT_ERR_UNSUPPORTED;
  if (c->d_ff % 4) return RT_ERR_UNSUPPORTED;
  if (B > kSmallBatchMax && !(wide_ok && c->sched == RT_SCHED_TILED)) return RT_ERR_UNSUPPORTED;
  return RT_OK;
}

WsLayout ws_layout(const rt_config* c, int B, int N) {
  WsLayout L;
  const size_t e = esize_of(c->dtype), d = c->d_model, H = c->n_heads, f = c->d_ff;
  const size_t tok = (size_t)B * N;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += align_up(bytes, 256); return at; };
  L.sync = take(sizeof(SyncArea));
  L.q = take(tok * d * e);
  L.kt = take(tok * d * e);
  L.vt = take(tok * d * e);
  L.n = take(tok * d * e);
  L.st_o = take(tok * d * 4);
  L.st_m = take(tok * H * 4);
  L.st_l = take(tok * H * 4);
  L.ex_h = take((size_t)B * d * 4);
  L.ex_g = take((size_t)B * f * 4);
  L.ex_z = take((size_t)B * d * 4);
  L.ex_k = take((size_t)B * d * 4);
  L.ex_part = take((size_t)B * H * kMaxChunks * 68 * 4);
  L.dec_part = take((size_t)B * H * kDecodeMaxRowChunks * 66 * 4);   // chunk partials of the decode-step attention
  // exchange buffers of the tensor-core leaf kernel: c, h, z as flag-carrying words (16 sequence slots each),
  // g as packed bf16 in fragment order (16 sequence slots), raw k|v as flag-carrying fp32 words
  L.ll_bytes = ((size_t)16 * 3 * (d / 2) + (size_t)16 * (f / 4) + (size_t)B * 2 * d) * 8;
  L.ll = take(L.ll_bytes);
  L.hid0 = take(tok * d * e);
  L.hid1 = take(tok * d * e);
  // recurrence over blocks: the position-wise chain of one block (rows = block length x B)
  L.blk_h = L.blk_u = L.blk_c = L.blk_g = 0;
  if (c->recur_block > 1) {
    const size_t rows = (size_t)B * (c->recur_block < N ? c->recur_block : N);
    L.blk_h = take(rows * d * 4);
    L.blk_u = take(rows * d * e);
    L.blk_c = take(rows * d * e);
    L.blk_g = take(rows * f * e);
  }
  L.total = o;
  return L;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b);
  return pa < pb + nb && pb < pa + na;
}

bool weights_ok(const rt_layer_weights* w) {
  if (!w) return false;
  const void* req[] = {w->w_q, w->w_k, w->w_v, w->w_o, w->w_up, w->w_down};
  for (const void* p : req) if (!p || !aligned16(p)) return false;
  const void* opt[] = {w->g_attn, w->g_mlp, w->g_kv, w->g_q, w->g_k};
  for (const void* p : opt) if (p && !aligned16(p)) return false;
  return true;
}

int leaf_size(const rt_config* c) { return c->leaf ? c->leaf : kAutoLeaf; }

// Which form of the per-token chain a prefill with this configuration and batch runs, and the granularity of
// Algorithm 1's tiles that goes with it.  Used by run_layer and by rt_plan_counters, so that the modelled schedule is
// the one that runs (the tensor-core leaf kernel's leaf depends on the shared memory of the part; the planner assumes
// a B200).
enum ChainPath { kPathGeneric = 0, kPathMma = 1, kPathWide = 2, kPathBlocks = 3, kPathMmaSplit = 4 };
struct Schedule { ChainPath path; int leaf; int sub; };      // sub: sequences per launch of the tensor-core leaf kernel (kPathMmaSplit)
constexpr int kWideLeafDefault = 16;    // leaf of the dense-product token steps: the in-leaf attention re-reads the leaf's pairs for every position,
                                        // so short leaves win (p512: 16 -> 41.6 ms, 32 -> 42.3, 64 -> 45.9 per layer)
constexpr int kMmaSplitMax = 48;         // largest batch that runs as slices of at most 16 sequences through the tensor-core leaf kernel
Schedule effective_schedule(const rt_config* c, int B) {
  if (c->recur_block > 1) return {kPathBlocks, c->recur_block, 0};
  if (c->sched == RT_SCHED_TILED) {
    LeafMmaLaunch ml;
    if (c->dtype == RT_BF16 && B > 16 && B <= kMmaSplitMax) {
      // Sequences are independent (Sec. 2.2 states the layer per sequence) and a token step of the tensor-core leaf
      // kernel costs 10 - 14 us whatever its batch, against 53 us for the dense-product step at B = 32: up to 48
      // sequences run as 2 or 3 slices of at most 16 through that kernel, leaf by leaf, and share the cross tiles.
      const int n_sub = (B + 15) / 16, sub = (B + n_sub - 1) / n_sub;
      if (leaf_mma_shape(sub, c->d_model, c->n_heads, c->d_ff, c->leaf, kB200Sms, kB200SmemPerCta, &ml))
        return {kPathMmaSplit, ml.leaf, sub};
    }
    // bf16 batches beyond that (or whose slices the tensor-core leaf kernel does not take) run as dense products from
    // 24 sequences on, where they overtake the generic kernel (measured at d = 1024: 53 us per token step at B = 32
    // against 99 us); fp32 keeps the generic kernel up to its limit
    if (B > kSmallBatchMax || (c->dtype == RT_BF16 && B >= 24)) return {kPathWide, c->leaf ? c->leaf : kWideLeafDefault, 0};
    if (c->dtype == RT_BF16 && leaf_mma_shape(B, c->d_model, c->n_heads, c->d_ff, c->leaf, kB200Sms, kB200SmemPerCta, &ml))
      return {kPathMma, ml.leaf, B};
  }
  return {kPathGeneric, leaf_size(c), 0};
}

// ---- optional per-kernel-class timing (rt_profile_enable / rt_profile_read) -----------------
enum ProfClass { kProfPrepass = 0, kProfLeaf = 1, kProfTile = 2, kProfOther = 3, kProfClasses = 4 };
struct ProfSpan { cudaEvent_t a, b; int cls; };
std::mutex g_prof_mu;
bool g_prof_on = false;
bool g_prof_timers = false;      // rt_profile_enable(2): also the in-kernel phase timers of the leaf kernels
std::vector<ProfSpan> g_prof_spans;
constexpr size_t kProfMaxSpans = 1u << 20;

// Records an event pair around the launches issued inside its scope when profiling is on.
struct ProfScope {
  cudaStream_t s; int cls; cudaEvent_t a = nullptr, b = nullptr; bool on = false;
  ProfScope(cudaStream_t s_, int cls_) : s(s_), cls(cls_) {
    std::lock_guard<std::mutex> g(g_prof_mu);
    if (!g_prof_on || g_prof_spans.size() >= kProfMaxSpans) return;
    if (cudaEventCreate(&a) != cudaSuccess) return;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return; }
    on = cudaEventRecord(a, s) == cudaSuccess;
  }
  ~ProfScope() {
    if (!a) return;
    if (on && cudaEventRecord(b, s) == cudaSuccess) {
      std::lock_guard<std::mutex> g(g_prof_mu);
      g_prof_spans.push_back({a, b, cls});
    } else { cudaEventDestroy(a); cudaEventDestroy(b); }
  }
};

// State of one API call: the stream and the barrier arrivals enqueued so far.
struct CallCtx { cudaStream_t s; unsigned bar_base = 0; unsigned seq_base = 0; };

// One layer on position-major scratch; x / z given with explicit strides.
rt_status run_layer(const rt_config* c, const rt_layer_weights* w, const void* x, long long x_bs, long long x_ts,
                    void* z, long long z_bs, long long z_ts, int B, int n_rows, int pos0, void* k_cache,
                    void* v_cache, int n_max, unsigned char* ws, const WsLayout& L, CallCtx& ctx) {
  // n_rows positions starting at cache position pos0 (prefill: pos0 = 0; decode: n_rows = 1)
  cudaStream_t s = ctx.s;
  const float scale_log2 = c->softmax_scale * kLog2e;
  PrepassParams pp;
  memset(&pp, 0, sizeof(pp));
  pp.B = B; pp.N = n_rows; pp.d = c->d_model; pp.H = c->n_heads;
  pp.norm_flags = c->norm_flags; pp.eps = c->rms_eps; pp.scale_log2 = scale_log2;
  pp.x = x; pp.x_bs = x_bs; pp.x_ts = x_ts;
  pp.w_q = w->w_q; pp.w_k = w->w_k; pp.w_v = w->w_v;
  pp.g_attn = w->g_attn; pp.g_q = w->g_q; pp.g_k = w->g_k;
  pp.n = ws + L.n; pp.q = ws + L.q; pp.kt = ws + L.kt; pp.vt = ws + L.vt;
  pp.st_o = (float*)(ws + L.st_o); pp.st_m = (float*)(ws + L.st_m); pp.st_l = (float*)(ws + L.st_l);
  pp.sync = (SyncArea*)(ws + L.sync);
  // decode step on the fast path (bf16 shapes the tensor-core leaf kernel takes): its attention warps seed the state
  LeafMmaLaunch ml;
  const bool dec_fast = n_rows == 1 && pos0 > 0 && c->dtype == RT_BF16 && c->recur_block <= 1 &&
                        leaf_mma_plan(B, c->d_model, c->n_heads, c->d_ff, c->leaf, &ml);
  if (dec_fast && (size_t)16 * (c->d_model + 16) * 2 <= 190 * 1024) {
    // the decode step's pre-pass in one launch (the leaf kernel's attention warps seed the state)
    DecodePrepassParams dp;
    memset(&dp, 0, sizeof(dp));
    dp.B = B; dp.d = c->d_model; dp.H = c->n_heads; dp.norm_flags = c->norm_flags; dp.eps = c->rms_eps;
    dp.x = x; dp.x_bs = x_bs;
    dp.w_q = w->w_q; dp.w_k = w->w_k; dp.w_v = w->w_v; dp.g_attn = w->g_attn; dp.g_q = w->g_q; dp.g_k = w->g_k;
    dp.q = pp.q; dp.kt = pp.kt; dp.vt = pp.vt;
    ProfScope ps(s, kProfPrepass);
    if (decode_prepass_launch(dp, s) != cudaSuccess) return RT_ERR_CUDA;
  } else {
    if (dec_fast) pp.no_seed = 1;
    ProfScope ps(s, kProfPrepass);
    if (prepass_launch(c->dtype, pp, s) != cudaSuccess) return RT_ERR_CUDA;
  }

  if (c->recur_block > 1) {
    // Recurrence over blocks of S positions: a block is one parallel sweep (in-block causal attention over the
    // TEMPORARY pairs, the position-wise chain as dense products over the block's rows, then its persistent pairs),
    // and blocks follow each other with Algorithm 1's cross tiles at block granularity.
    if (c->sched != RT_SCHED_TILED || pos0 != 0) return RT_ERR_UNSUPPORTED;
    const int S = c->recur_block, N = n_rows;
    const long long d = c->d_model, f = c->d_ff;
    const size_t e = esize_of(c->dtype);
    SyncArea* sync = (SyncArea*)(ws + L.sync);
    const bool pre = (c->norm_flags & RT_NORM_PRE) != 0;
    TileParams tp;
    memset(&tp, 0, sizeof(tp));
    tp.B = B; tp.d = c->d_model; tp.H = c->n_heads; tp.scale_log2 = scale_log2; tp.alibi = w->alibi_slopes;
    tp.q = ws + L.q; tp.st_o = pp.st_o; tp.st_m = pp.st_m; tp.st_l = pp.st_l;
    tp.rows_q = n_rows; tp.sync = sync;
    PrepassParams pk = pp;                                      // persistent pairs of a block from its outputs
    pk.x_bs = z_bs; pk.x_ts = z_ts;
    pk.norm_flags = (c->norm_flags & RT_NORM_SKIP_Z) ? (c->norm_flags & ~RT_NORM_PRE) : c->norm_flags;
    pk.g_attn = w->g_kv ? w->g_kv : w->g_attn;
    pk.mats = 6; pk.no_seed = 1; pk.chained = 1;              // the chain of a block: programmatic dependent launches
    DenseParams dp;
    memset(&dp, 0, sizeof(dp));
    dp.chained = 1;
    dp.B = B; dp.alpha = c->residual_scale; dp.h = (float*)(ws + L.blk_h);
    const int Lb = c->dtype == RT_BF16 ? 2 * kAutoLeaf : kAutoLeaf;
    for (int s0 = 0; s0 < N; s0 += S) {
      const int e0 = s0 + S < N ? s0 + S : N, rows = e0 - s0;
      {
        // 1. in-block attention over the temporary pairs of strictly earlier positions (the pair of the position
        //    itself is in the seeded state): causal diagonal blocks, then the levels inside the block
        ProfScope ps(s, kProfTile);
        tp.k_cache = ws + L.kt; tp.v_cache = ws + L.vt; tp.rows_kv = n_rows; tp.q_limit = e0;
        const int full = rows / Lb;
        tp.causal = 1;
        if (c->dtype == RT_BF16 && rows % Lb == 0 && rows >= 4 * Lb) {
          // whole blocks of 128, tensor cores: every query's causal prefix inside the block in one launch
          tp.q0 = s0; tp.q1 = e0; tp.k0 = s0; tp.k1 = e0; tp.batch = 0; tp.batch_stride = 0; tp.causal_full = 1;
          if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
          tp.causal_full = 0;
        } else {
          if (full > 0) {
            tp.q0 = s0; tp.q1 = s0 + Lb; tp.k0 = s0; tp.k1 = s0 + Lb; tp.batch = full; tp.batch_stride = Lb;
            if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
          }
          if (full * Lb < rows) {
            tp.q0 = s0 + full * Lb; tp.q1 = e0; tp.k0 = tp.q0; tp.k1 = e0; tp.batch = 1; tp.batch_stride = 0;
            if (tile_simt_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
          }
          tp.causal = 0;
          for (long long P = Lb; P < rows; P *= 2) {
            tp.q0 = s0 + (int)P; tp.q1 = s0 + (int)(2 * P); tp.k0 = s0; tp.k1 = s0 + (int)P;
            tp.batch = (int)((rows - P + 2 * P - 1) / (2 * P)); tp.batch_stride = (int)(2 * P);
            if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
          }
        }
        tp.causal = 0; tp.batch = 0; tp.batch_stride = 0; tp.q_limit = 0;
      }
      {
        // 2. position-wise chain over the block's rows, 3. its persistent pairs
        ProfScope ps(s, kProfLeaf);
        const size_t row = (size_t)s0 * B;
        void* cbuf = ws + L.blk_c; void* ubuf = ws + L.blk_u; void* gbuf = ws + L.blk_g;
        if (attn_value_launch(c->dtype, pp.st_o + row * d, pp.st_l + row * c->n_heads, cbuf, (long long)rows * B, (int)d, c->n_heads, s, true) != cudaSuccess)
          return RT_ERR_CUDA;
        dp.M = rows * B;
        dp.N = (int)d; dp.K = (int)d; dp.A = cbuf; dp.W = w->w_o; dp.epi = DENSE_RES_X;
        dp.x = (const unsigned char*)x + (size_t)s0 * x_ts * e; dp.x_bs = x_bs; dp.x_ts = x_ts;
        if (dense_launch(c->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
        if (rms_rows_f32_launch(c->dtype, dp.h, w->g_mlp, ubuf, rows * B, (int)d, c->rms_eps, pre ? 1 : 0, s, true) != cudaSuccess) return RT_ERR_CUDA;
        dp.N = (int)f; dp.K = (int)d; dp.A = ubuf; dp.W = w->w_up; dp.epi = DENSE_GELU; dp.out = gbuf;
        if (dense_launch(c->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
        dp.N = (int)d; dp.K = (int)f; dp.A = gbuf; dp.W = w->w_down; dp.epi = DENSE_RES_H;
        dp.out = (unsigned char*)z + (size_t)s0 * z_ts * e; dp.o_bs = z_bs; dp.o_ts = z_ts;
        if (dense_launch(c->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
        pk.N = rows;
        pk.x = (const unsigned char*)z + (size_t)s0 * z_ts * e;
        pk.kt = (unsigned char*)k_cache + row * d * e; pk.vt = (unsigned char*)v_cache + row * d * e;
        if (prepass_launch(c->dtype, pk, s) != cudaSuccess) return RT_ERR_CUDA;
      }
      if (e0 < N) {
        // 4. Algorithm 1 at block granularity: the next P positions attend to the last P persistent pairs
        const int u = e0 / S;
        const long long P = (long long)S * (u & -u);
        tp.k_cache = k_cache; tp.v_cache = v_cache; tp.rows_kv = n_max;
        tp.q0 = e0; tp.q1 = e0 + P < N ? (int)(e0 + P) : N; tp.k0 = (int)(e0 - P); tp.k1 = e0;
        ProfScope ps(s, kProfTile);
        if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
      }
    }
    return RT_OK;
  }

  const Schedule plan = effective_schedule(c, B);
  const bool wide = B > kSmallBatchMax || (plan.path == kPathWide && pos0 == 0);
  if (wide) {
    // Wide batches (the regime of the paper's own experiments, Sec. 6: B in the hundreds): a token step is a chain
    // of dense products with M = B rows, so it runs on the tensor cores through the same kernels as the parallel
    // sweep, one position at a time; the schedule (leaf, then the cross tile of Algorithm 1) is unchanged.
    if (c->sched != RT_SCHED_TILED || pos0 != 0) return RT_ERR_UNSUPPORTED;
    const long long d = c->d_model, f = c->d_ff;
    const size_t e = esize_of(c->dtype);
    SyncArea* sync = (SyncArea*)(ws + L.sync);
    float* hbuf = (float*)(ws + L.ex_h);                        // [B, d] fp32
    void* gbuf = ws + L.ex_g;                                   // [B, d_ff] storage type
    void* ubuf = ws + L.ex_z;                                   // [B, d] storage type
    void* cbuf = ws + L.ex_k;                                   // [B, d] storage type
    const bool pre = (c->norm_flags & RT_NORM_PRE) != 0;
    TileParams tp;
    memset(&tp, 0, sizeof(tp));
    tp.B = B; tp.d = c->d_model; tp.H = c->n_heads; tp.scale_log2 = scale_log2; tp.alibi = w->alibi_slopes;
    tp.q = ws + L.q; tp.k_cache = k_cache; tp.v_cache = v_cache;
    tp.st_o = pp.st_o; tp.st_m = pp.st_m; tp.st_l = pp.st_l;
    tp.rows_q = n_rows; tp.rows_kv = n_max; tp.sync = sync;
    PrepassParams pk = pp;                                      // persistent pair of one position from its output
    pk.N = 1; pk.x_bs = z_bs; pk.x_ts = z_ts;
    pk.norm_flags = (c->norm_flags & RT_NORM_SKIP_Z) ? (c->norm_flags & ~RT_NORM_PRE) : c->norm_flags;
    pk.g_attn = w->g_kv ? w->g_kv : w->g_attn;
    pk.mats = 6; pk.no_seed = 1;
    // the seven launches of a token step are short and strictly dependent: chained (programmatic dependent
    // launches), each is scheduled while its predecessor drains
    pk.chained = 1; tp.chained = 1;
    DenseParams dp;
    memset(&dp, 0, sizeof(dp));
    dp.chained = 1;
    dp.M = B; dp.B = B; dp.alpha = c->residual_scale; dp.h = hbuf;
    dp.partial = (float*)(ws + L.ex_part); dp.partial_bytes = (size_t)B * c->n_heads * kMaxChunks * 68 * 4;
    // in-leaf attention re-reads the leaf's pairs for every position (leaf^2 * B * d bytes per leaf), so wide
    // batches default to a shorter leaf
    const int Lf = plan.path == kPathWide ? plan.leaf : (c->leaf ? c->leaf : kWideLeafDefault), N = n_rows;
    for (int s0 = 0; s0 < N; s0 += Lf) {
      const int e0 = s0 + Lf < N ? s0 + Lf : N;
      {
        ProfScope ps(s, kProfLeaf);
        for (int t = s0; t < e0; ++t) {
          // pairs of this leaf revealed so far (none for its first position), then c = o / l of the finished row
          tp.q0 = t; tp.q1 = t + 1; tp.k0 = s0; tp.k1 = t; tp.c_out = cbuf;
          if (row_attn_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
          tp.c_out = nullptr;
          const size_t row = (size_t)t * B;
          bool normed = false;
          dp.N = (int)d; dp.K = (int)d; dp.A = cbuf; dp.W = w->w_o; dp.epi = DENSE_RES_X;
          dp.x = (const unsigned char*)x + (size_t)t * x_ts * e; dp.x_bs = x_bs; dp.x_ts = 0;
          dp.norm_out = ubuf; dp.norm_gain = w->g_mlp; dp.norm_eps = c->rms_eps; dp.norm_pre = pre ? 1 : 0;   // u = RMS(h)
          if (dense_launch(c->dtype, dp, sync, s, &normed) != cudaSuccess) return RT_ERR_CUDA;
          if (!normed && rms_rows_f32_launch(c->dtype, hbuf, w->g_mlp, ubuf, B, (int)d, c->rms_eps, pre ? 1 : 0, s, true) != cudaSuccess)
            return RT_ERR_CUDA;
          dp.norm_out = nullptr;
          dp.N = (int)f; dp.K = (int)d; dp.A = ubuf; dp.W = w->w_up; dp.epi = DENSE_GELU; dp.out = gbuf;
          if (dense_launch(c->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
          dp.N = (int)d; dp.K = (int)f; dp.A = gbuf; dp.W = w->w_down; dp.epi = DENSE_RES_H;
          dp.out = (unsigned char*)z + (size_t)t * z_ts * e; dp.o_bs = z_bs; dp.o_ts = 0;
          dp.norm_out = pk.n; dp.norm_gain = pk.g_attn; dp.norm_pre = (pk.norm_flags & RT_NORM_PRE) ? 1 : 0;          // RMS(z)
          if (dense_launch(c->dtype, dp, sync, s, &normed) != cudaSuccess) return RT_ERR_CUDA;
          dp.norm_out = nullptr;
          pk.skip_rms = normed ? 1 : 0;
          pk.x = (const unsigned char*)z + (size_t)t * z_ts * e;
          pk.kt = (unsigned char*)k_cache + row * d * e; pk.vt = (unsigned char*)v_cache + row * d * e;
          if (prepass_launch(c->dtype, pk, s) != cudaSuccess) return RT_ERR_CUDA;
        }
      }
      if (e0 < N) {
        const int P = e0 & -e0;
        tp.q0 = e0; tp.q1 = e0 + P < N ? e0 + P : N; tp.k0 = e0 - P; tp.k1 = e0;
        ProfScope ps(s, kProfTile);
        if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
      }
    }
    return RT_OK;
  }

  LeafLaunch ll;
  if (leaf_plan(c->dtype, B, c->d_model, c->d_ff, &ll) != cudaSuccess) return RT_ERR_CUDA;
  LeafParams lp;
  memset(&lp, 0, sizeof(lp));
  lp.B = B; lp.d = c->d_model; lp.H = c->n_heads; lp.dff = c->d_ff;
  lp.norm_flags = c->norm_flags; lp.eps = c->rms_eps; lp.scale_log2 = scale_log2; lp.alpha = c->residual_scale;
  lp.w_o = w->w_o; lp.w_up = w->w_up; lp.w_down = w->w_down; lp.w_k = w->w_k; lp.w_v = w->w_v;
  lp.g_mlp = w->g_mlp; lp.g_kv = w->g_kv ? w->g_kv : w->g_attn; lp.g_k = w->g_k; lp.alibi = w->alibi_slopes;
  lp.x = x; lp.x_bs = x_bs; lp.x_ts = x_ts;
  lp.z = z; lp.z_bs = z_bs; lp.z_ts = z_ts;
  lp.k_cache = k_cache; lp.v_cache = v_cache;
  lp.q = ws + L.q;
  lp.st_o = pp.st_o; lp.st_m = pp.st_m; lp.st_l = pp.st_l;
  lp.row_off = pos0;
  lp.ex_h = (float*)(ws + L.ex_h); lp.ex_g = (float*)(ws + L.ex_g);
  lp.ex_z = (float*)(ws + L.ex_z); lp.ex_k = (float*)(ws + L.ex_k);
  lp.ex_part = (float*)(ws + L.ex_part);
  lp.max_chunks = kMaxChunks;
  lp.timers = g_prof_timers ? 1 : 0;
  lp.sync = (SyncArea*)(ws + L.sync);

  auto leaf = [&](int t0, int t1, int attn_begin) -> bool {
    lp.t0 = t0; lp.t1 = t1; lp.attn_begin = attn_begin; lp.bar_base = ctx.bar_base;
    ProfScope ps(s, kProfLeaf);
    if (leaf_launch(c->dtype, lp, ll, s) != cudaSuccess) return false;
    ctx.bar_base += leaf_barrier_arrivals(t0, t1, ll.grid);
    return true;
  };

  // bf16 tiled prefill takes the tensor-core leaf kernel when the shape fits it
  // (batches of 17 .. 48 sequences: in slices of at most 16, see effective_schedule)
  const int b_sub = (plan.path == kPathMmaSplit && pos0 == 0) ? plan.sub : B;
  const bool use_mma = c->dtype == RT_BF16 && c->sched == RT_SCHED_TILED && pos0 == 0 &&
                       leaf_mma_plan(b_sub, c->d_model, c->n_heads, c->d_ff, c->leaf, &ml);
  LeafMmaBuffers mb;
  {
    unsigned long long* w = (unsigned long long*)(ws + L.ll);
    const size_t bd2 = (size_t)16 * (c->d_model / 2);
    mb.ll_c = w; mb.ll_h = w + bd2; mb.ll_z = w + 2 * bd2; mb.ll_g = w + 3 * bd2;
    mb.ll_kv = mb.ll_g + (size_t)16 * (c->d_ff / 4);
  }
  auto leaf_mma = [&](int t0, int t1) -> bool {
    ProfScope ps(s, kProfLeaf);
    const size_t e = esize_of(c->dtype);
    for (int b0 = 0; b0 < B; b0 += b_sub) {
      lp.B = B - b0 < b_sub ? B - b0 : b_sub; lp.Bs = B; lp.b0 = b0;
      lp.x = (const unsigned char*)x + (size_t)b0 * x_bs * e;
      lp.z = (unsigned char*)z + (size_t)b0 * z_bs * e;
      lp.t0 = t0; lp.t1 = t1; lp.attn_begin = t0; lp.seq_base = ctx.seq_base; lp.bar_base = ctx.bar_base;
      if (leaf_mma_launch(lp, ml, mb, s) != cudaSuccess) return false;
      ctx.seq_base += (unsigned)(t1 - t0);
      ctx.bar_base += (unsigned)(t1 - t0) * (unsigned)ml.grid;    // one grid barrier per token step
    }
    return true;
  };

  if (dec_fast) {
    // decode step on the fast path: the new position's query attends to the whole cache in chunks (Algorithm 2 per
    // chunk), then the tensor-core leaf kernel merges the partial states and runs the one token step
    DecodeAttnParams da;
    memset(&da, 0, sizeof(da));
    da.B = B; da.d = c->d_model; da.H = c->n_heads; da.scale_log2 = scale_log2; da.alibi = w->alibi_slopes;
    da.q = ws + L.q; da.k_cache = k_cache; da.v_cache = v_cache; da.pos = pos0;
    da.part = (float*)(ws + L.dec_part);
    int n_chunks = 0, chunk_stride = 0;
    {
      ProfScope ps(s, kProfTile);
      if (decode_attn_launch(da, &n_chunks, &chunk_stride, s) != cudaSuccess) return RT_ERR_CUDA;
    }
    lp.kt = ws + L.kt; lp.vt = ws + L.vt; lp.dec_part = da.part; lp.dec_chunks = n_chunks; lp.dec_stride = chunk_stride;
    lp.t0 = pos0; lp.t1 = pos0 + 1; lp.attn_begin = pos0; lp.seq_base = ctx.seq_base; lp.bar_base = ctx.bar_base;
    ProfScope ps(s, kProfLeaf);
    if (leaf_mma_launch(lp, ml, mb, s) != cudaSuccess) return RT_ERR_CUDA;
    ctx.seq_base += 1u;
    ctx.bar_base += (unsigned)ml.grid;
    return RT_OK;
  }
  if (c->sched == RT_SCHED_NAIVE || pos0 > 0) {
    // token-sequential: every position reads its whole prefix from the cache
    return leaf(pos0, pos0 + n_rows, 0) ? RT_OK : RT_ERR_CUDA;
  }
  TileParams tp;
  memset(&tp, 0, sizeof(tp));
  tp.B = B; tp.d = c->d_model; tp.H = c->n_heads; tp.scale_log2 = scale_log2; tp.alibi = w->alibi_slopes;
  tp.q = ws + L.q; tp.k_cache = k_cache; tp.v_cache = v_cache;
  tp.st_o = pp.st_o; tp.st_m = pp.st_m; tp.st_l = pp.st_l;
  tp.rows_q = n_rows; tp.rows_kv = n_max; tp.sync = lp.sync;
  const int Lf = use_mma ? ml.leaf : leaf_size(c), N = n_rows;
  for (int s0 = 0; s0 < N; s0 += Lf) {
    const int e0 = s0 + Lf < N ? s0 + Lf : N;
    if (!(use_mma ? leaf_mma(s0, e0) : leaf(s0, e0, s0))) return RT_ERR_CUDA;
    if (e0 < N) {
      const int P = e0 & -e0;                              // largest power of two dividing the block end
      tp.q0 = e0; tp.q1 = e0 + P < N ? e0 + P : N; tp.k0 = e0 - P; tp.k1 = e0;
      ProfScope ps(s, kProfTile);
      if (tile_launch(c->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
    }
  }
  return RT_OK;
}

rt_status common_checks(const rt_config* c, int B, int N, int n_layers, void* ws, size_t ws_bytes, bool wide_ok = false) {
  if (!config_ok(c) || B <= 0 || N <= 0 || n_layers <= 0 || !ws || !aligned16(ws)) return RT_ERR_INVALID_ARG;
  const rt_status st = config_supported(c, B, wide_ok);
  if (st != RT_OK) return st;
  // the recurrence over blocks exists for tiled prefill only (wide_ok marks the prefill entry points)
  if (c->recur_block > 1 && !(wide_ok && c->sched == RT_SCHED_TILED)) return RT_ERR_UNSUPPORTED;
  if (ws_bytes < ws_layout(c, B, N).total) return RT_ERR_WORKSPACE;
  return RT_OK;
}

}  // namespace

namespace rt {
ProfSpanScope::ProfSpanScope(cudaStream_t s, int cls) { impl = new ProfScope(s, cls); }
ProfSpanScope::~ProfSpanScope() { delete static_cast<ProfScope*>(impl); }
}  // namespace rt

extern "C" {

size_t rt_workspace_bytes(const rt_config* cfg, int32_t B, int32_t N, int32_t n_layers) {
  if (!config_ok(cfg) || B <= 0 || N <= 0 || n_layers <= 0) return 0;
  return ws_layout(cfg, B, N).total;
}

rt_status rt_layer_prefill(const rt_config* cfg, const rt_layer_weights* w, const void* x, int32_t B, int32_t N,
                           void* z, void* k_cache, void* v_cache, int32_t N_max, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
  rt_status st = common_checks(cfg, B, N, 1, workspace, workspace_bytes, true);
  if (st != RT_OK) return st;
  if (!weights_ok(w) || !x || !z || !k_cache || !v_cache || N_max < N) return RT_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(z) || !aligned16(k_cache) || !aligned16(v_cache)) return RT_ERR_INVALID_ARG;
  const size_t xz_bytes = (size_t)B * N * cfg->d_model * esize_of(cfg->dtype);
  if (overlaps(x, xz_bytes, z, xz_bytes)) return RT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)workspace;
  const WsLayout L = ws_layout(cfg, B, N);
  if (cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  if (cudaMemsetAsync(ws + L.ll, 0, L.ll_bytes, s) != cudaSuccess) return RT_ERR_CUDA;
  const long long d = cfg->d_model;
  CallCtx ctx{s};
  return run_layer(cfg, w, x, (long long)N * d, d, z, (long long)N * d, d, B, N, 0, k_cache, v_cache, N_max, ws, L, ctx);
}

size_t rt_recompute_workspace_bytes(const rt_config* cfg, int32_t B, int32_t N) {
  if (!config_ok(cfg) || B <= 0 || N <= 0) return 0;
  return ws_layout(cfg, B, N).total + align_up((size_t)B * N * cfg->d_ff * esize_of(cfg->dtype), 256);
}

rt_status rt_layer_recompute(const rt_config* cfg, const rt_layer_weights* w, const void* x, const void* z_claim,
                             int32_t B, int32_t N, void* z_out, void* k_cache, void* v_cache, int32_t N_max,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!config_ok(cfg) || B <= 0 || N <= 0 || !workspace || !aligned16(workspace)) return RT_ERR_INVALID_ARG;
  rt_status st = config_supported(cfg, 1);
  if (st != RT_OK) return st;
  if (cfg->recur_block > 1) return RT_ERR_UNSUPPORTED;          // the sweep is the fixed-point map of the layer of Sec. 2.2
  if (workspace_bytes < rt_recompute_workspace_bytes(cfg, B, N)) return RT_ERR_WORKSPACE;
  if (!weights_ok(w) || !x || !z_claim || !z_out || !k_cache || !v_cache || z_out == x || z_out == z_claim || N_max < N)
    return RT_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(z_claim) || !aligned16(z_out) || !aligned16(k_cache) || !aligned16(v_cache))
    return RT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)workspace;
  const WsLayout L = ws_layout(cfg, B, N);
  if (cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  const long long d = cfg->d_model, f = cfg->d_ff;
  const long long tok = (long long)B * N;
  const float scale_log2 = cfg->softmax_scale * kLog2e;
  SyncArea* sync = (SyncArea*)(ws + L.sync);
  const bool pre = (cfg->norm_flags & RT_NORM_PRE) != 0;

  // 1. every persistent pair from the claimed outputs (Eqs. 1-2): k = qkRMS[W_k RMS(z)], v = W_v RMS(z)
  PrepassParams pz;
  memset(&pz, 0, sizeof(pz));
  pz.B = B; pz.N = N; pz.d = cfg->d_model; pz.H = cfg->n_heads;
  pz.norm_flags = (cfg->norm_flags & RT_NORM_SKIP_Z) ? (cfg->norm_flags & ~RT_NORM_PRE) : cfg->norm_flags;
  pz.eps = cfg->rms_eps; pz.scale_log2 = scale_log2;
  pz.x = z_claim; pz.x_bs = (long long)N * d; pz.x_ts = d;
  pz.w_q = w->w_q; pz.w_k = w->w_k; pz.w_v = w->w_v;
  pz.g_attn = w->g_kv ? w->g_kv : w->g_attn; pz.g_q = w->g_q; pz.g_k = w->g_k;
  pz.n = ws + L.n; pz.q = ws + L.q; pz.kt = k_cache; pz.vt = v_cache;
  pz.st_o = (float*)(ws + L.st_o); pz.st_m = (float*)(ws + L.st_m); pz.st_l = (float*)(ws + L.st_l);
  pz.mats = 6; pz.no_seed = 1; pz.sync = sync;
  {
    ProfScope ps(s, kProfPrepass);
    if (prepass_launch(cfg->dtype, pz, s) != cudaSuccess) return RT_ERR_CUDA;
  }
  // 2. queries, temporary pairs and the seeded running stats from the layer input, as in the prefill
  PrepassParams px = pz;
  px.norm_flags = cfg->norm_flags;
  px.x = x; px.g_attn = w->g_attn;
  px.kt = ws + L.kt; px.vt = ws + L.vt;
  px.mats = 0; px.no_seed = 0;
  {
    ProfScope ps(s, kProfPrepass);
    if (prepass_launch(cfg->dtype, px, s) != cudaSuccess) return RT_ERR_CUDA;
  }
  // 3. attention of every query over all earlier persistent pairs: the pairs inside a 64-block under a causal
  //    mask, then Algorithm 1's cross tiles, one launch per level (all pairs are known, so the tiles of a level are
  //    independent; each query row meets exactly one tile per level)
  TileParams tp;
  memset(&tp, 0, sizeof(tp));
  tp.B = B; tp.d = cfg->d_model; tp.H = cfg->n_heads; tp.scale_log2 = scale_log2; tp.alibi = w->alibi_slopes;
  tp.q = ws + L.q; tp.k_cache = k_cache; tp.v_cache = v_cache;
  tp.st_o = px.st_o; tp.st_m = px.st_m; tp.st_l = px.st_l;
  tp.rows_q = N; tp.rows_kv = N_max; tp.sync = sync; tp.q_limit = N;
  {
    ProfScope ps(s, kProfTile);
    // diagonal blocks under the causal mask: whole blocks in one batched launch (tensor cores for bf16), the
    // ragged last block on its own; then the levels of Algorithm 1 from the block size upwards
    const int Lb = cfg->dtype == RT_BF16 ? 2 * kAutoLeaf : kAutoLeaf;
    const int full = N / Lb;
    tp.causal = 1;
    if (cfg->dtype == RT_BF16 && N % Lb == 0 && N >= 4 * Lb) {
      // whole blocks only, tensor cores: every query's causal prefix in ONE launch (a CTA walks over the key blocks up to
      // its own query tile) instead of diagonal blocks plus one launch per level of short tiles
      tp.q0 = 0; tp.q1 = N; tp.k0 = 0; tp.k1 = N; tp.batch = 0; tp.batch_stride = 0; tp.causal_full = 1;
      if (tile_launch(cfg->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
      tp.causal_full = 0; tp.causal = 0;
      goto attention_done;
    }
    if (full > 0) {
      tp.q0 = 0; tp.q1 = Lb; tp.k0 = 0; tp.k1 = Lb; tp.batch = full; tp.batch_stride = Lb;
      if (tile_launch(cfg->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
    }
    if (full * Lb < N) {
      tp.q0 = full * Lb; tp.q1 = N; tp.k0 = full * Lb; tp.k1 = N; tp.batch = 1; tp.batch_stride = 0;
      if (tile_simt_launch(cfg->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
    }
    tp.causal = 0;
    for (long long P = Lb; P < N; P *= 2) {
      tp.q0 = (int)P; tp.q1 = (int)(2 * P); tp.k0 = 0; tp.k1 = (int)P;
      tp.batch = (int)((N - P + 2 * P - 1) / (2 * P)); tp.batch_stride = (int)(2 * P);
      if (tile_launch(cfg->dtype, tp, s) != cudaSuccess) return RT_ERR_CUDA;
    }
  attention_done:;
  }
  // 4. position-wise chain over all rows at once
  ProfScope ps(s, kProfOther);
  void* cbuf = ws + L.kt;                                       // the temporary pairs are folded into the stats by now
  void* ubuf = ws + L.vt;
  float* hbuf = (float*)(ws + L.st_o);                          // free once c = o / l is taken
  void* gbuf = ws + L.total;
  if (attn_value_launch(cfg->dtype, px.st_o, px.st_l, cbuf, tok, (int)d, cfg->n_heads, s) != cudaSuccess) return RT_ERR_CUDA;
  DenseParams dp;
  memset(&dp, 0, sizeof(dp));
  dp.M = (int)tok; dp.B = B; dp.alpha = cfg->residual_scale; dp.h = hbuf;
  dp.N = (int)d; dp.K = (int)d; dp.A = cbuf; dp.W = w->w_o; dp.epi = DENSE_RES_X;
  dp.x = x; dp.x_bs = (long long)N * d; dp.x_ts = d;
  if (dense_launch(cfg->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
  if (rms_rows_f32_launch(cfg->dtype, hbuf, w->g_mlp, ubuf, (int)tok, (int)d, cfg->rms_eps, pre ? 1 : 0, s) != cudaSuccess)
    return RT_ERR_CUDA;
  dp.N = (int)f; dp.K = (int)d; dp.A = ubuf; dp.W = w->w_up; dp.epi = DENSE_GELU; dp.out = gbuf;
  if (dense_launch(cfg->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
  dp.N = (int)d; dp.K = (int)f; dp.A = gbuf; dp.W = w->w_down; dp.epi = DENSE_RES_H;
  dp.out = z_out; dp.o_bs = (long long)N * d; dp.o_ts = d;
  if (dense_launch(cfg->dtype, dp, sync, s) != cudaSuccess) return RT_ERR_CUDA;
  return RT_OK;
}

rt_status rt_layer_decode_step(const rt_config* cfg, const rt_layer_weights* w, const void* x, int32_t B, int32_t pos,
                               void* z, void* k_cache, void* v_cache, int32_t N_max, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
  rt_status st = common_checks(cfg, B, 1, 1, workspace, workspace_bytes);
  if (st != RT_OK) return st;
  if (!weights_ok(w) || !x || !z || !k_cache || !v_cache || pos < 0 || pos >= N_max) return RT_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(z) || !aligned16(k_cache) || !aligned16(v_cache)) return RT_ERR_INVALID_ARG;
  {
    const size_t xz_bytes = (size_t)B * cfg->d_model * esize_of(cfg->dtype);
    if (overlaps(x, xz_bytes, z, xz_bytes)) return RT_ERR_INVALID_ARG;
  }
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)workspace;
  const WsLayout L = ws_layout(cfg, B, 1);
  if (cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  if (cudaMemsetAsync(ws + L.ll, 0, L.ll_bytes, s) != cudaSuccess) return RT_ERR_CUDA;
  const long long d = cfg->d_model;
  rt_config c = *cfg;
  c.sched = RT_SCHED_NAIVE;
  CallCtx ctx{s};
  return run_layer(&c, w, x, d, d, z, d, d, B, 1, pos, k_cache, v_cache, N_max, ws, L, ctx);
}

rt_status rt_stack_prefill(const rt_config* cfg, int32_t n_layers, const rt_layer_weights* layers, const void* emb,
                           const void* g_final, int32_t vocab, const int32_t* ids, int32_t B, int32_t N, void* hidden,
                           float* logits_last, void* const* k_caches, void* const* v_caches, int32_t N_max,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
  rt_status st = common_checks(cfg, B, N, n_layers, workspace, workspace_bytes, true);
  if (st != RT_OK) return st;
  if (!layers || !emb || !ids || !k_caches || !v_caches || vocab <= 0 || N_max < N) return RT_ERR_INVALID_ARG;
  if (!aligned16(emb) || (hidden && !aligned16(hidden)) || (g_final && !aligned16(g_final))) return RT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!weights_ok(&layers[l]) || !k_caches[l] || !v_caches[l] || !aligned16(k_caches[l]) || !aligned16(v_caches[l]))
      return RT_ERR_INVALID_ARG;
  }
  if ((size_t)B * cfg->d_model * 4 > 200 * 1024) return RT_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)workspace;
  const WsLayout L = ws_layout(cfg, B, N);
  if (cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  if (cudaMemsetAsync(ws + L.ll, 0, L.ll_bytes, s) != cudaSuccess) return RT_ERR_CUDA;
  const long long d = cfg->d_model;
  void* bufs[2] = {ws + L.hid0, ws + L.hid1};
  CallCtx ctx{s};
  {
    ProfScope ps(s, kProfOther);
    if (embed_launch(cfg->dtype, emb, ids, B, N, (int)d, vocab, bufs[0], s) != cudaSuccess) return RT_ERR_CUDA;
  }
  const void* cur = bufs[0];
  for (int l = 0; l < n_layers; ++l) {
    void* out = (l == n_layers - 1 && hidden) ? hidden : bufs[(l + 1) & 1];
    st = run_layer(cfg, &layers[l], cur, (long long)N * d, d, out, (long long)N * d, d, B, N, 0, k_caches[l],
                   v_caches[l], N_max, ws, L, ctx);
    if (st != RT_OK) return st;
    cur = out;
  }
  if (logits_last) {
    ProfScope ps(s, kProfOther);
    const unsigned char* last = (const unsigned char*)cur + (size_t)(N - 1) * d * esize_of(cfg->dtype);
    if (head_launch(cfg->dtype, emb, g_final, last, (long long)N * d, B, (int)d, vocab, cfg->norm_flags, cfg->rms_eps,
                    logits_last, s) != cudaSuccess)
      return RT_ERR_CUDA;
  }
  return RT_OK;
}

rt_status rt_decode_step(const rt_config* cfg, int32_t n_layers, const rt_layer_weights* layers, const void* emb,
                         const void* g_final, int32_t vocab, const int32_t* ids, int32_t B, int32_t pos, float* logits,
                         void* const* k_caches, void* const* v_caches, int32_t N_max, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  rt_status st = common_checks(cfg, B, 1, n_layers, workspace, workspace_bytes);
  if (st != RT_OK) return st;
  if (!layers || !emb || !ids || !logits || !k_caches || !v_caches || vocab <= 0 || pos < 0 || pos >= N_max)
    return RT_ERR_INVALID_ARG;
  if (!aligned16(emb) || (g_final && !aligned16(g_final))) return RT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!weights_ok(&layers[l]) || !k_caches[l] || !v_caches[l] || !aligned16(k_caches[l]) || !aligned16(v_caches[l]))
      return RT_ERR_INVALID_ARG;
  }
  if ((size_t)B * cfg->d_model * 4 > 200 * 1024) return RT_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)workspace;
  const WsLayout L = ws_layout(cfg, B, 1);
  if (cudaMemsetAsync(ws + L.sync, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  if (cudaMemsetAsync(ws + L.ll, 0, L.ll_bytes, s) != cudaSuccess) return RT_ERR_CUDA;
  const long long d = cfg->d_model;
  rt_config c = *cfg;
  c.sched = RT_SCHED_NAIVE;
  void* bufs[2] = {ws + L.hid0, ws + L.hid1};
  CallCtx ctx{s};
  if (embed_launch(c.dtype, emb, ids, B, 1, (int)d, vocab, bufs[0], s) != cudaSuccess) return RT_ERR_CUDA;
  const void* cur = bufs[0];
  for (int l = 0; l < n_layers; ++l) {
    void* out = bufs[(l + 1) & 1];
    st = run_layer(&c, &layers[l], cur, d, d, out, d, d, B, 1, pos, k_caches[l], v_caches[l], N_max, ws, L, ctx);
    if (st != RT_OK) return st;
    cur = out;
  }
  if (head_launch(c.dtype, emb, g_final, cur, d, B, (int)d, vocab, c.norm_flags, c.rms_eps, logits, s) != cudaSuccess)
    return RT_ERR_CUDA;
  return RT_OK;
}

rt_status rt_get_status(const void* workspace) {
  if (!workspace) return RT_ERR_INVALID_ARG;
  int st = 0;
  if (cudaMemcpy(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RT_ERR_CUDA;
  return (rt_status)st;
}

rt_status rt_update_tile(const rt_config* cfg, const void* q, const void* k_cache, const void* v_cache, float* st_o,
                         float* st_m, float* st_l, int32_t B, int32_t rows_q, int32_t rows_kv, int32_t q0, int32_t q1,
                         int32_t k0, int32_t k1, const float* alibi_slopes, void* workspace, void* cuda_stream) {
  if (!config_ok(cfg) || B <= 0 || !q || !k_cache || !v_cache || !st_o || !st_m || !st_l || !workspace)
    return RT_ERR_INVALID_ARG;
  if (q0 < 0 || q1 < q0 || q1 > rows_q || k0 < 0 || k1 < k0 || k1 > rows_kv) return RT_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(st_o) || !aligned16(workspace))
    return RT_ERR_INVALID_ARG;
  const rt_status sup = config_supported(cfg, B, true);        // a tile takes any batch
  if (sup != RT_OK) return sup;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (cudaMemsetAsync(workspace, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  TileParams tp;
  memset(&tp, 0, sizeof(tp));
  tp.B = B; tp.d = cfg->d_model; tp.H = cfg->n_heads; tp.scale_log2 = cfg->softmax_scale * kLog2e; tp.alibi = alibi_slopes;
  tp.q = q; tp.k_cache = k_cache; tp.v_cache = v_cache;
  tp.st_o = st_o; tp.st_m = st_m; tp.st_l = st_l;
  tp.q0 = q0; tp.q1 = q1; tp.k0 = k0; tp.k1 = k1;
  tp.rows_q = rows_q; tp.rows_kv = rows_kv; tp.sync = (SyncArea*)workspace;
  ProfScope ps(s, kProfTile);
  return tile_launch(cfg->dtype, tp, s) == cudaSuccess ? RT_OK : RT_ERR_CUDA;
}

rt_status rt_selftest_wait_expiry(void* workspace, void* cuda_stream) {
  if (!workspace || !aligned16(workspace)) return RT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (cudaMemsetAsync(workspace, 0, sizeof(SyncArea), s) != cudaSuccess) return RT_ERR_CUDA;
  return wait_expiry_selftest_launch((SyncArea*)workspace, s) == cudaSuccess ? RT_OK : RT_ERR_CUDA;
}

rt_status rt_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> g(g_prof_mu);
  g_prof_on = on != 0;
  g_prof_timers = on >= 2;
  return RT_OK;
}

rt_status rt_profile_read(rt_profile* out) {
  if (!out) return RT_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  std::vector<ProfSpan> spans;
  {
    std::lock_guard<std::mutex> g(g_prof_mu);
    spans.swap(g_prof_spans);
  }
  rt_status st = RT_OK;
  for (const ProfSpan& sp : spans) {
    float ms = 0.f;
    if (cudaEventSynchronize(sp.b) != cudaSuccess || cudaEventElapsedTime(&ms, sp.a, sp.b) != cudaSuccess) st = RT_ERR_CUDA;
    else { out->ms[sp.cls] += ms; out->launches[sp.cls] += 1; }
    cudaEventDestroy(sp.a);
    cudaEventDestroy(sp.b);
  }
  return st;
}

const char* rt_status_string(rt_status s) {
  switch (s) {
    case RT_OK: return "ok";
    case RT_ERR_INVALID_ARG: return "invalid argument";
    case RT_ERR_UNSUPPORTED: return "unsupported configuration";
    case RT_ERR_WORKSPACE: return "workspace too small";
    case RT_ERR_CUDA: return "CUDA runtime error";
    case RT_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int32_t rt_plan_tiles(int32_t N, int32_t leaf, int32_t* out, int32_t cap) {
  if (N <= 0 || leaf <= 0) return 0;
  int32_t n = 0;
  for (int s0 = 0; s0 < N; s0 += leaf) {
    const int e0 = s0 + leaf < N ? s0 + leaf : N;
    if (e0 >= N) break;
    const int blocks = e0 / leaf;
    const int P = leaf * (blocks & -blocks);
    if (out && n < cap) {
      out[4 * n + 0] = e0; out[4 * n + 1] = e0 + P < N ? e0 + P : N;
      out[4 * n + 2] = e0 - P; out[4 * n + 3] = e0;
    }
    ++n;
  }
  return n;
}

rt_status rt_plan_counters(const rt_config* cfg, int32_t B, int32_t N, int32_t n_layers, int32_t vocab,
                           rt_counters* out) {
  if (!config_ok(cfg) || B <= 0 || N <= 0 || n_layers <= 0 || vocab < 0 || !out) return RT_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  const uint64_t e = esize_of(cfg->dtype), d = cfg->d_model, H = cfg->n_heads, f = cfg->d_ff, b = B, n = N;
  const uint64_t tok = b * n;
  uint64_t rd = 0, wr = 0, kv = 0, kv_leaf = 0, fl_tile = 0, fl_leaf = 0, tiles = 0, leaves = 0;
  // pre-pass: RMS (x -> n), projection (n, W -> q, k~, v~), state seed (q, k~, v~ -> o, m, l)
  rd += tok * d * e + tok * d * e + 3 * d * d * e + 3 * tok * d * e;
  wr += tok * d * e + 3 * tok * d * e + tok * d * 4 + 2 * tok * H * 4;
  const uint64_t chain_w = (3 * d * d + 2 * d * f) * e;
  // per token: q row, carried state, x row in; z, k, v rows out
  rd += tok * d * e + tok * (d + 2 * H) * 4 + tok * d * e;
  wr += 3 * tok * d * e;
  fl_leaf += tok * 2 * (3 * d * d + 2 * d * f);
  if (cfg->sched == RT_SCHED_NAIVE) {
    leaves = 1;
    rd += chain_w;
    kv = b * d * e * n * (n - 1);                        // K and V rows of the whole prefix, every position
    fl_leaf += 4 * d * b * (n * (n - 1) / 2);
  } else {
    // the schedule that runs: leaf (or block) granularity of the chain form this shape takes
    const Schedule plan = effective_schedule(cfg, B);
    const uint64_t Lf = plan.leaf;
    for (uint64_t s0 = 0; s0 < n; s0 += Lf) {
      const uint64_t e0 = s0 + Lf < n ? s0 + Lf : n, len = e0 - s0;
      ++leaves;
      // persistent kernels stage their weight rows once per leaf launch; dense products (wide batches, block sweeps)
      // stream them once per position resp. once per block
      rd += chain_w * (plan.path == kPathWide ? len : (plan.path == kPathMmaSplit ? (b + plan.sub - 1) / plan.sub : 1));
      kv_leaf += 2 * b * d * e * (len * (len - 1) / 2);  // in-leaf pairs: written a few steps earlier, L2-resident
      fl_leaf += 4 * d * b * (len * (len - 1) / 2);
      if (e0 < n) {
        const uint64_t blocks = e0 / Lf;
        const uint64_t P = Lf * (blocks & (~blocks + 1));
        const uint64_t nq = (e0 + P < n ? e0 + P : n) - e0;
        ++tiles;
        kv += 2 * P * b * d * e;
        rd += nq * b * d * e + nq * b * (d + 2 * H) * 4;
        wr += nq * b * (d + 2 * H) * 4;
        fl_tile += 4 * nq * P * d * b;
      }
    }
  }
  rd += kv;
  out->model_bytes_read = rd * n_layers;
  out->model_bytes_written = wr * n_layers;
  out->kv_bytes_read = kv * n_layers;
  out->leaf_kv_bytes_l2 = kv_leaf * n_layers;
  out->flops_tile = fl_tile * n_layers;
  out->flops_leaf = fl_leaf * n_layers;
  out->flops_gemm = tok * 2 * d * 3 * d * n_layers;
  out->n_tiles = tiles * n_layers;
  out->n_leaves = leaves * n_layers;
  if (vocab > 0) {
    out->model_bytes_read += tok * d * e + (uint64_t)vocab * d * e;
    out->model_bytes_written += tok * d * e + b * (uint64_t)vocab * 4;
    out->flops_gemm += 2 * b * d * (uint64_t)vocab;
  }
  return RT_OK;
}

}  // extern "C"
