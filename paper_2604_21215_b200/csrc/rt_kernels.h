// Host-side launch interface of the RT kernels (internal; the public ABI is include/rt.h).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "rt_common.cuh"

namespace rt {

// Everything the per-token chain needs.  Position-major buffers are [row, B, d] with
// row = t - row_off (prefill: row_off = 0; decode: the single row 0 stands for position pos).
struct LeafParams {
  int B, d, H, dff;
  int norm_flags;
  float eps, scale_log2, alpha;
  const void *w_o, *w_up, *w_down, *w_k, *w_v;   // storage type
  const void *g_mlp, *g_kv, *g_k;                // storage type or NULL
  const float* alibi;                            // [H] slopes of the ALiBi distances (natural-log units) or NULL
  const void* x;  long long x_bs, x_ts;          // x[b, t, :] = x + b*x_bs + (t-row_off)*x_ts   (elements)
  void* z;        long long z_bs, z_ts;
  void *k_cache, *v_cache;                       // [N_max, B, d] storage type
  const void* q;                                 // [rows, B, d] storage type
  float *st_o, *st_m, *st_l;                     // online-softmax state: o [rows,B,d], m,l [rows,B,H] (m in log2 units)
  int t0, t1;                                    // positions [t0, t1) are processed by this launch
  int row_off;
  // tensor-core leaf kernel on a slice of the batch: the rows of q, the state and the caches are [row][Bs][...] and this
  // launch's sequence b is column b0 + b of them (x and z are passed already offset); Bs = 0 means Bs = B, b0 = 0
  int Bs, b0;
  int attn_begin;                                // first key position the in-launch attention covers (0 = whole prefix)
  float *ex_h, *ex_g, *ex_z, *ex_k;              // exchange vectors [B,d], [B,dff], [B,d], [B,d]
  float* ex_part;                                // partial attention states [B*H, max_chunks, 66]
  int max_chunks;
  int weights_in_smem;                           // 1: each CTA keeps its weight rows in shared memory
  unsigned bar_base;                             // arrivals counted by earlier launches of the same call (bar_count is
                                                 // zeroed once per API call and only ever grows)
  unsigned seq_base;                             // token steps enqueued before this launch in the same call (flag values)
  // decode step through the tensor-core leaf kernel (one position): the attention warps build the position's state
  // themselves -- seeded with the temporary pair (kt, vt rows [B, d]), then the cache's chunk partials
  // ([B*H][dec_chunks][66] floats: o, m, l) folded in chunk order; dec_chunks = 0 otherwise
  const void *kt, *vt;
  const float* dec_part;
  int dec_chunks, dec_stride;
  int timers;                                    // 1: CTA 0 accumulates per-phase times in the sync area (costs a few per cent)
  SyncArea* sync;
};

struct LeafLaunch { int grid, block; size_t smem; int weights_in_smem; };

// Chooses grid / shared memory for the leaf kernel on the current device.
cudaError_t leaf_plan(int dtype, int B, int d, int dff, LeafLaunch* out);
cudaError_t leaf_launch(int dtype, const LeafParams& p, const LeafLaunch& l, cudaStream_t s);
// Barrier arrivals one launch over [t0,t1) adds to bar_count.
inline unsigned leaf_barrier_arrivals(int t0, int t1, int grid) { return (unsigned)(t1 - t0) * 5u * (unsigned)grid; }

// launches a 2-CTA kernel whose barrier cannot complete (tests the bounded-wait path)
cudaError_t wait_expiry_selftest_launch(SyncArea* sync, cudaStream_t s);

// bf16 / tiled-schedule leaf kernel (tensor-core mat-vecs, flag-carrying exchange words).
struct LeafMmaLaunch { int grid, block; size_t smem; int leaf; int q_smem; };
struct LeafMmaBuffers { unsigned long long *ll_c, *ll_h, *ll_g, *ll_z, *ll_kv; };   // [16,d/2] words x3, packed bf16 [B,dff], [B,2d] words
bool leaf_mma_plan(int B, int d, int H, int dff, int want_leaf, LeafMmaLaunch* out);
// the same decision for a device with `sms` multiprocessors and `max_smem` bytes of shared memory per CTA (no CUDA call)
bool leaf_mma_shape(int B, int d, int H, int dff, int want_leaf, int sms, size_t max_smem, LeafMmaLaunch* out);
constexpr int kB200Sms = 148;                    // the part this library is written for: what the pure-host planner assumes
constexpr size_t kB200SmemPerCta = 232448;
cudaError_t leaf_mma_launch(const LeafParams& p, const LeafMmaLaunch& l, const LeafMmaBuffers& buf, cudaStream_t s);

// Pre-pass (Algorithm 1, line 1 and the temporary pair of line 7, hoisted out of the loop).
struct PrepassParams {
  int B, N, d, H;
  int norm_flags;
  float eps, scale_log2;
  const void* x; long long x_bs, x_ts;           // x[b, r, :]
  const void *w_q, *w_k, *w_v, *g_attn, *g_q, *g_k;
  void* n;                                       // [N*B, d] normalised input (scratch)
  void *q, *kt, *vt;                             // [N, B, d]
  float *st_o, *st_m, *st_l;
  int mats;                                      // which projections to compute: bit 0 q, bit 1 k, bit 2 v (0 = all three)
  int no_seed;                                   // 1: leave the running stats alone (projection only)
  int skip_rms;                                  // 1: `n` already holds the normalised rows
  int chained;                                   // 1: launch the projection as a programmatic dependent launch
  SyncArea* sync;
};
cudaError_t prepass_launch(int dtype, const PrepassParams& p, cudaStream_t s);
// tensor-core projection (bf16, d a multiple of 128)
bool qkv_gemm_tc_supported(const PrepassParams& p);
cudaError_t qkv_gemm_tc_launch(const PrepassParams& p, SyncArea* sync, cudaStream_t s);

// Cross-block tile (Algorithm 2 on a [q0,q1) x [k0,k1) block for every sequence and head).
struct TileParams {
  int B, d, H;
  float scale_log2;
  const float* alibi;                            // [H] slopes of the ALiBi distances (natural-log units) or NULL
  const void* q;                                 // [N, B, d]
  const void *k_cache, *v_cache;                 // [N_max, B, d]
  float *st_o, *st_m, *st_l;
  int q0, q1, k0, k1;
  int batch, batch_stride, q_limit;              // batch > 1: blockIdx.z-th copy of the tile, shifted by z * batch_stride rows
                                                 // (one level of Algorithm 1 in one launch); q_limit > 0 clips the queries
  int causal;                                    // 1: only pairs with key position < query position
  int causal_full;                               // with causal (tensor-core kernel): a CTA's key blocks end at its own query tile, so one
                                                 // launch over [q0,q1) x [k0,k1) covers every query's whole causal prefix; heavy tiles first
  int chained;                                   // row_attn only: launch as a programmatic dependent launch
  void* c_out;                                   // row_attn only: also write the attention value o/l of the row, [B, d] storage type
  int rows_q, rows_kv;                           // rows held by the query buffer / the caches (tensor-map bounds)
  SyncArea* sync;
};
cudaError_t tile_launch(int dtype, const TileParams& p, cudaStream_t s);
// tensor-core version (bf16, key count a multiple of 64)
cudaError_t tile_tc_launch(const TileParams& p, int rows_q, int rows_kv, SyncArea* sync, cudaStream_t s);
cudaError_t tile_simt_launch(int dtype, const TileParams& p, cudaStream_t s);
// one query row (position q0) per (sequence, head) against the pairs [k0, k1): the in-leaf step of wide batches
cudaError_t row_attn_launch(int dtype, const TileParams& p, cudaStream_t s);

// Attention of one decode step over the whole cache (bf16): query row q [B, d] of the new position against the pairs
// [0, pos), chunk partials (o, m, l) in `part` ([B*H][n_chunks][66] floats, n_chunks <= kDecodeMaxChunks); the leaf
// kernel's attention warps fold them, in chunk order, into the state seeded with the temporary pair.
constexpr int kDecodeMaxChunks = 64;
constexpr int kDecodeMaxRowChunks = 320;         // chunks of the long-cache kernel (its partials are merged to one per pair)
struct DecodeAttnParams {
  int B, d, H;
  float scale_log2;
  const float* alibi;                            // [H] slopes or NULL
  const void* q;                                 // [B, d] bf16
  const void *k_cache, *v_cache;                 // [N_max, B, d] bf16
  int pos;                                       // positions in the cache
  int chunk, n_chunks;                           // set by the launcher
  float* part;
};
// Launches the partial kernel(s); *n_chunks = partial states per (sequence, head) left for the leaf kernel to fold in,
// *chunk_stride = slots per pair in `part` (the leaf kernel reads slots 0 .. n_chunks-1 of pair u at u * chunk_stride).
cudaError_t decode_attn_launch(const DecodeAttnParams& p, int* n_chunks, int* chunk_stride, cudaStream_t s);

// Pre-pass of a decode step (bf16, B <= 16, d a multiple of 16 with 16 (d + 16) 2 bytes of shared memory available):
// n = RMS(x), q, k~, v~ of the one new row per sequence in one launch; x [B, d] with row stride x_bs, outputs [B, d].
struct DecodePrepassParams {
  int B, d, H;
  int norm_flags;
  float eps;
  const void* x; long long x_bs;
  const void *w_q, *w_k, *w_v, *g_attn, *g_q, *g_k;
  void *q, *kt, *vt;
};
cudaError_t decode_prepass_launch(const DecodePrepassParams& p, cudaStream_t s);

// Stack helpers.
cudaError_t embed_launch(int dtype, const void* emb, const int32_t* ids, int B, int N, int d, int vocab,
                         void* x, cudaStream_t s);
cudaError_t head_launch(int dtype, const void* emb, const void* g_final, const void* hidden, long long h_bs,
                        int B, int d, int vocab, int norm_flags, float eps, float* logits, cudaStream_t s);

// Position-wise part of the parallel sweep (Sec. 6, activation checkpointing): dense products over all rows.
enum { DENSE_RES_X = 0, DENSE_GELU = 1, DENSE_RES_H = 2, DENSE_F32 = 3 };
struct DenseParams {
  int M, N, K, B;                                // C[M,N] = A[M,K] W[N,K]^T; rows m = position * B + sequence
  const void *A, *W;                             // storage type, K contiguous
  int epi;                                       // DENSE_RES_X: h = x + alpha C (fp32);  DENSE_GELU: out = GELU(C);
                                                 // DENSE_RES_H: out = h + alpha C (storage type, caller's strides)
                                                 // DENSE_F32: h = alpha C, or h += alpha C with `accumulate` (fp32 [M, N])
  float alpha;
  int accumulate;                                // DENSE_F32 only
  const void* x; long long x_bs, x_ts;           // x[b, r, :] (DENSE_RES_X)
  float* h;                                      // [M, N] fp32 (written by DENSE_RES_X, read by DENSE_RES_H)
  void* out; long long o_bs, o_ts;               // DENSE_GELU: [M, N];  DENSE_RES_H: out[b, r, :]
  float* partial; size_t partial_bytes;          // optional scratch for a split contraction (few rows): [splits, M, N] fp32
  int splits;                                    // set by the launcher
  int chained;                                   // 1: launch the product (and its reduction) as programmatic dependent launches
  // optional: also write RMS_g(row) of the epilogue's result (h or z) for the next product.  Only a split
  // contraction does this (its reduction kernel owns whole rows); `normed` tells the caller whether it happened.
  void* norm_out; const void* norm_gain; float norm_eps; int norm_pre;
  // DENSE_QKV (persistent CTA pairs only): three products A W_q^T, A W_k^T, A W_v^T in one launch, N = d columns each;
  // qkRMS over each head's 64 columns of q and k (qk_norm), bf16 outputs [M, d]
  const void *W2, *W3;                           // W = W_q, W2 = W_k, W3 = W_v
  void *q_out, *k_out, *v_out;
  const void *g_q, *g_k;
  int qk_norm; float qk_eps;
};
constexpr int DENSE_QKV = 100;
// The q / k~ / v~ projections of the pre-pass as one launch of persistent CTA pairs (bf16, d a multiple of 256, at least a
// wave of tiles); false when the shape does not qualify (the caller then takes qkv_gemm_tc_launch's own kernel).
bool dense_qkv_pair_supported(int M, int d);
cudaError_t dense_qkv_pair_launch(const DenseParams& p, SyncArea* sync, cudaStream_t s);
cudaError_t dense_launch(int dtype, const DenseParams& p, SyncArea* sync, cudaStream_t s, bool* normed = nullptr);
cudaError_t attn_value_launch(int dtype, const float* st_o, const float* st_l, void* c, long long rows, int d, int H, cudaStream_t s,
                              bool chained = false);
cudaError_t rms_rows_f32_launch(int dtype, const float* h, const void* g, void* u, int rows, int d, float eps, int pre, cudaStream_t s,
                                bool chained = false);

// Event-pair span for rt_profile_enable / rt_profile_read from other translation units (classes: 0 sweeps / pre-pass,
// 1 per-position steps, 2 attention tiles, 3 everything else).  Does nothing while profiling is off.
struct ProfSpanScope {
  void* impl = nullptr;
  ProfSpanScope(cudaStream_t s, int cls);
  ~ProfSpanScope();
  ProfSpanScope(const ProfSpanScope&) = delete;
  ProfSpanScope& operator=(const ProfSpanScope&) = delete;
};

}  // namespace rt
