/*
 * rt.h -- C ABI of the B200 (sm_100a) Recurrent Transformer prefill library.
 *
 * The library evaluates, exactly, the Recurrent Transformer (RT) layer of Sec. 2.2 of
 * "The Recurrent Transformer" (arXiv 2604.21215): at position i the query and a TEMPORARY
 * key/value pair come from the layer input x_i, the attention runs over the PERSISTENT
 * pairs of earlier positions plus that temporary pair, the layer output is
 *     z_i = x_i + alpha (a_i + MLP[RMS(x_i + alpha a_i)]),
 * and the persistent pair of position i is computed from z_i (Eqs. 1-2).  Prefill uses
 * the exact tiling schedule of Sec. 5 / Algorithms 1-2 (App. C).
 *
 * Conventions for every entry point
 *  - All tensor pointers are DEVICE pointers unless a comment says "host".  The caller owns
 *    every buffer, including the workspace; the library allocates no device memory.  Its only
 *    state outside the caller's buffers: the profiling switch (rt_profile_enable), the built-in
 *    scratch array of rt_layer_decode_step_static, and per-thread caches of encoded tensor maps
 *    and kernel attributes (pure functions of their arguments).  It reads no environment
 *    variables.  Pointers must be 16-byte aligned.
 *  - Storage type (rt_dtype) applies to x, weights, gains, z, the K/V caches and the
 *    embedding.  Accumulation is always fp32.  Logits are fp32.
 *  - Weights are row-major [out, in]:  y = W u.
 *  - x and z are [B, N, d_model] row-major.  z must not overlap x (checked: RT_ERR_INVALID_ARG).
 *  - A K/V cache is POSITION-MAJOR [N_max, B, d_model] (Sec. 6, "Cache locality"): row t
 *    holds the persistent pair of position t for all sequences.  Prefill writes rows [0, N),
 *    decode appends row pos.  All sequences of a batch share the same length.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL = default
 *    stream) and return without synchronising.  Argument, shape, alignment and workspace
 *    errors, and configurations an entry point does not support, are detected on the host
 *    before anything is enqueued.  A device-side bounded
 *    wait that runs out is recorded in the workspace and read with rt_get_status after the
 *    caller has synchronised the stream.  Nothing aborts, traps or throws.
 *  - The same workspace must not be used by two calls that overlap in time.
 */
#ifndef RT_B200_H
#define RT_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RT_OK = 0,
  RT_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, misaligned pointer, inconsistent shape */
  RT_ERR_UNSUPPORTED = 2,   /* valid request this build has no kernel for (e.g. head_dim != 64) */
  RT_ERR_WORKSPACE = 3,     /* workspace_bytes < rt_workspace_bytes(...) */
  RT_ERR_CUDA = 4,          /* a CUDA runtime call failed (launch, attribute query) */
  RT_ERR_TIMEOUT = 5        /* a bounded device-side wait expired; outputs are invalid */
} rt_status;

typedef enum { RT_F32 = 0, RT_BF16 = 1 } rt_dtype;

/* RT_SCHED_TILED: Algorithm 1's schedule at leaf granularity (each K/V row is streamed
 * O(log N) times).  RT_SCHED_NAIVE: the token-sequential evaluation of Sec. 5 ("What makes
 * naive evaluation slow"): every position reads its whole prefix, Theta(N^2) traffic; kept
 * as the comparison path.  Both give the same result up to rounding order. */
typedef enum { RT_SCHED_TILED = 0, RT_SCHED_NAIVE = 1 } rt_sched;

enum {                      /* rt_config.norm_flags (bit 2 is not used: Sec. 2.2 normalises queries and keys "independently
                               per head", and a full-width variant would need a reduction across all heads inside every
                               token step of the leaf kernel; any other bit is RT_ERR_INVALID_ARG) */
  RT_NORM_PRE = 1,          /* RMS(x_i), RMS before the MLP and RMS(z_i) are applied (Sec. 2.2) */
  RT_NORM_QK = 2,           /* qkRMS on queries and keys, per head */
  RT_NORM_SKIP_Z = 8        /* persistent pair from z_i itself (the RMSNorm-ablation appendix) */
};

enum {                      /* rt_config.flags */
  RT_FLAG_BACKWARD_STEP_LAUNCHES = 1   /* rt_layer_backward: run the reverse loop as one launch per step instead of one
                                          cooperative launch per leaf (the form a device without cooperative launch gets
                                          anyway; same device code, used by tests to compare the two) */
};

typedef struct {
  int32_t d_model, n_heads, head_dim, d_ff; /* n_heads*head_dim == d_model; head_dim must be 64 */
  int32_t dtype;            /* rt_dtype */
  int32_t sched;            /* rt_sched */
  int32_t leaf;             /* leaf block size of the tiled schedule: power of two in [16, 256]; 0 = auto */
  int32_t norm_flags;       /* RT_NORM_*; the paper's layer is RT_NORM_PRE | RT_NORM_QK */
  float rms_eps;            /* added to the mean square inside the root (the paper gives none; 1e-6) */
  float softmax_scale;      /* logits = scale * <q, k>.  Sec. 2's Attn has scale 1; 1/sqrt(head_dim) is customary */
  float residual_scale;     /* alpha = 1/sqrt(L) of Sec. 2; 1 for a single layer */
  int32_t recur_block;      /* 0 or 1: the layer of Sec. 2.2.  S > 1: recurrence over blocks of S positions (Sec. 9 names this
                               extension without defining it; the reading taken: position i attends to the persistent pairs
                               of all positions in earlier blocks and to the temporary pairs of the positions j <= i of its own
                               block, so a block is computed in one parallel sweep; S >= N is an ordinary pre-LN Transformer
                               layer).  Prefill entry points only, tiled schedule; decode returns RT_ERR_UNSUPPORTED */
  int32_t flags;            /* RT_FLAG_*; 0 for the defaults */
} rt_config;

typedef struct {            /* device pointers; read-only */
  const void *w_q, *w_k, *w_v, *w_o;   /* [d_model, d_model]; w_k and w_v serve the temporary AND the persistent pair */
  const void *w_up;                    /* [d_ff, d_model] */
  const void *w_down;                  /* [d_model, d_ff]   MLP(u) = w_down GELU(w_up u), exact (erf) GELU, no biases */
  const void *g_attn, *g_mlp, *g_kv;   /* [d_model] RMS gains of RMS(x), the MLP pre-norm and RMS(z); NULL = ones; g_kv NULL = g_attn */
  const void *g_q, *g_k;               /* [d_model] qkRMS gains; NULL = ones */
  const float *alibi_slopes;           /* [n_heads] fp32, or NULL for none.  ALiBi distances (App. D: the paper's experiments
                                          use them, maximum bias 8): the logit of query i on the persistent pair of position j
                                          gets -alibi_slopes[h] * (i - j); the temporary pair of position i sits at distance 0 */
} rt_layer_weights;

/* Bytes of workspace a call with these shapes needs (N = positions per call: the prefill
 * length, or 1 for decode).  n_layers >= 1.  Returns 0 for an invalid configuration. */
size_t rt_workspace_bytes(const rt_config *cfg, int32_t B, int32_t N, int32_t n_layers);

/* One RT layer over x[B,N,d] (Sec. 2.2; Algorithm 1).  Writes z[B,N,d] and rows [0,N) of
 * k_cache / v_cache [N_max,B,d] (Eqs. 1-2).  N_max >= N.
 * Batch sizes (tiled schedule): B <= 16 in bf16 takes the persistent tensor-core leaf kernel; 17 <= B <= 48 in bf16
 * runs as 2 or 3 slices of at most 16 sequences through that kernel, leaf by leaf (the sequences are independent),
 * sharing the pre-pass and the cross tiles; larger batches run each token step as dense products over the batch
 * (bf16 from B = 49, fp32 from B = 65: the regime of the paper's own experiments, Sec. 6).  fp32 up to B = 64, the
 * naive schedule and decode up to B = 64 take a generic kernel.
 * The naive schedule and the decode entry points return RT_ERR_UNSUPPORTED for B > 64. */
rt_status rt_layer_prefill(const rt_config *cfg, const rt_layer_weights *w,
                           const void *x, int32_t B, int32_t N,
                           void *z, void *k_cache, void *v_cache, int32_t N_max,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* A stack of n_layers RT layers with token embedding and tied output head:
 * x^0 = emb[ids], x^l = layer_l(x^{l-1}), logits = emb . RMS_{g_final}(x^L at the last position).
 * `layers`, `k_caches`, `v_caches` are HOST arrays of n_layers entries (device pointers inside).
 * hidden [B,N,d] (storage type) and logits_last [B,vocab] (fp32) may each be NULL.
 * The head keeps one fp32 row of d_model per sequence in shared memory: B * d_model * 4 bytes must not exceed 200 KB
 * (RT_ERR_UNSUPPORTED otherwise; the same holds for rt_decode_step). */
rt_status rt_stack_prefill(const rt_config *cfg, int32_t n_layers, const rt_layer_weights *layers,
                           const void *emb, const void *g_final, int32_t vocab,
                           const int32_t *ids, int32_t B, int32_t N,
                           void *hidden, float *logits_last,
                           void *const *k_caches, void *const *v_caches, int32_t N_max,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One decode step of the stack: one new token id per sequence at position `pos` (the
 * number of positions already in the caches).  A forward pass of RT is a sequence of such
 * steps (Sec. 5), so this equals prefill of pos+1 tokens at its last position.  Appends row
 * pos to every cache; writes logits [B,vocab] (fp32). */
rt_status rt_decode_step(const rt_config *cfg, int32_t n_layers, const rt_layer_weights *layers,
                         const void *emb, const void *g_final, int32_t vocab,
                         const int32_t *ids, int32_t B, int32_t pos,
                         float *logits, void *const *k_caches, void *const *v_caches, int32_t N_max,
                         void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Decode step of a single layer: x[B,d] at position pos -> z[B,d]; appends row pos. */
rt_status rt_layer_decode_step(const rt_config *cfg, const rt_layer_weights *w,
                               const void *x, int32_t B, int32_t pos,
                               void *z, void *k_cache, void *v_cache, int32_t N_max,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The single-layer decode step for callers that cannot allocate device memory (the paper has
 * no counterpart: this is a packaging variant of rt_layer_decode_step, same arithmetic).
 * Meant for hosts that are handed their input and output buffers and nothing else, that run
 * where cudaMalloc is forbidden (it synchronises the device), or whose memory is fully
 * committed to K/V caches.  Instead of a caller-owned workspace it uses a scratch array of
 * RT_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the library
 * holds those bytes until the process exits.
 *  - x, z, k_cache, v_cache, N_max, pos: exactly as for rt_layer_decode_step.
 *  - Shapes whose rt_workspace_bytes(cfg, B, 1, 1) exceeds RT_STATIC_SCRATCH_BYTES are rejected
 *    with RT_ERR_WORKSPACE before anything is enqueued.
 *  - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - The first call on a device looks up the scratch array's device address (with that device
 *    current); make that first call before any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's contents; the
 *    words that must start from zero are cleared on the stream at the start of each call.  Two
 *    calls that overlap on the GPU (different streams, no dependency) race on it: serialise them.
 *  - The device status word of such a call lives in the built-in scratch: read it with
 *    rt_static_get_status() (below) after synchronising the stream. */
#define RT_STATIC_SCRATCH_BYTES (8u << 20)
rt_status rt_layer_decode_step_static(const rt_config *cfg, const rt_layer_weights *w,
                                      const void *x, int32_t B, int32_t pos,
                                      void *z, void *k_cache, void *v_cache, int32_t N_max,
                                      void *cuda_stream);

/* rt_get_status for the built-in scratch of rt_layer_decode_step_static on the current device (the paper has no
 * counterpart): after the caller synchronised the stream, copies back the status word of the last such call
 * (a blocking 4-byte copy): RT_OK, or RT_ERR_TIMEOUT when a bounded device-side wait ran out.  Allocates nothing. */
rt_status rt_static_get_status(void);

/* After the caller synchronised the stream: copies the device status word of `workspace`
 * back (a blocking 4-byte copy) and returns it (RT_OK or RT_ERR_TIMEOUT). */
rt_status rt_get_status(const void *workspace);

const char *rt_status_string(rt_status s);

/* Modelled work of the schedule that a prefill with these shapes runs (pure host function,
 * no CUDA call): bytes each launch is designed to move between HBM and the SMs, and flops.
 * vocab = 0 for a single layer fed with x. */
typedef struct {
  uint64_t model_bytes_read, model_bytes_written;
  uint64_t flops_tile;      /* cross-block tiles: 4 * queries * keys * head_dim per head */
  uint64_t flops_leaf;      /* per-token chain and in-leaf attention */
  uint64_t flops_gemm;      /* Q / temporary K,V projection (and the head, if vocab > 0) */
  uint64_t kv_bytes_read;   /* part of model_bytes_read: K/V cache rows streamed by the cross tiles (or, naive, by every position) */
  uint64_t leaf_kv_bytes_l2; /* NOT in model_bytes_read: rows of a position's own leaf, re-read while still L2-resident */
  uint64_t n_tiles, n_leaves;
} rt_counters;
rt_status rt_plan_counters(const rt_config *cfg, int32_t B, int32_t N, int32_t n_layers, int32_t vocab,
                           rt_counters *out);

/* Algorithm 2 (UpdateTile, App. C) on its own: queries [q0,q1) of `q` attend to the pairs [k0,k1) of
 * the caches, for every sequence and head, and their running stats are updated in place:
 *   m_new = max(m, max_j a_ij),  o = o*e^(m-m_new) + sum_j v_j e^(a_ij-m_new),  l likewise,  m = m_new,
 * with a_ij = softmax_scale <q_i, k_j> - alibi_slopes[h] * (i - j)  (rows of q and of the caches are positions;
 * alibi_slopes [n_heads] fp32 on the device, or NULL for no distance term).  The library keeps m in log2 units:
 * st_m holds log2(e)*m.
 * q [rows_q, B, d] and the caches [rows_kv, B, d] are position-major, storage type; st_o [rows_q, B, d],
 * st_m, st_l [rows_q, B, n_heads] are fp32.  `workspace` needs 256 bytes (device status word, read with
 * rt_get_status).  This is the cross-block step of rt_layer_prefill, exposed for tests and benchmarks. */
rt_status rt_update_tile(const rt_config *cfg, const void *q, const void *k_cache, const void *v_cache,
                         float *st_o, float *st_m, float *st_l,
                         int32_t B, int32_t rows_q, int32_t rows_kv,
                         int32_t q0, int32_t q1, int32_t k0, int32_t k1,
                         const float *alibi_slopes, void *workspace, void *cuda_stream);

/* One parallel sweep over all positions (Sec. 6, "activation checkpointing": with the layer outputs known, the
 * persistent pairs of all positions can be rebuilt at once and every position recomputed independently).
 * Given the layer input x [B,N,d] and claimed outputs z_claim [B,N,d]:
 *   k_j = qkRMS[W_k RMS(z_claim_j)], v_j = W_v RMS(z_claim_j)            -> k_cache, v_cache rows [0,N)  (Eqs. 1-2)
 *   a_i = attention of q_i over the pairs j < i and its temporary pair;  z'_i = x_i + alpha (a_i + MLP[RMS(x_i + alpha a_i)])
 *                                                                         -> z_out [B,N,d]
 * Because z_i depends only on z_j, j < i, the true outputs are the unique fixed point: z_out equals z_claim (up to
 * rounding) exactly when z_claim is what rt_layer_prefill returns.  All products run over the B*N rows at once
 * (tensor cores for bf16 storage), the attention as one causal pass inside 64-blocks plus one launch per level of
 * Algorithm 1.  x, z_claim, z_out are distinct buffers; the workspace needs rt_recompute_workspace_bytes. */
size_t    rt_recompute_workspace_bytes(const rt_config *cfg, int32_t B, int32_t N);
rt_status rt_layer_recompute(const rt_config *cfg, const rt_layer_weights *w, const void *x, const void *z_claim,
                             int32_t B, int32_t N, void *z_out, void *k_cache, void *v_cache, int32_t N_max,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Backward pass of one layer (Sec. 6, "The backward pass" and "activation checkpointing").
 * Inputs: the layer input x [B,N,d] and its outputs z [B,N,d] as rt_layer_prefill returned them (storage type; z is the
 * next layer's input, so a training loop keeps it anyway), and dz = dL/dz [B,N,d] fp32.
 * Outputs: dx = dL/dx [B,N,d] fp32 and the parameter gradients in `grads` (fp32, device, shapes of the parameters,
 * OVERWRITTEN; 16-byte aligned; a NULL entry is skipped; the entry of a gain the layer does not have (NULL in `w`) is set to zero).
 * When w->g_kv is NULL the gain of RMS(z) IS g_attn, and grads->g_attn carries both uses.
 * The call first rebuilds every intermediate from x and z in one parallel sweep, then walks the positions in reverse
 * accumulating only d(k_j, v_j) -- position i needs dL/dz_i, which needs d(k_i, v_i) complete; pairs in other leaves
 * of 64 positions receive their share from Algorithm 1's tiles run backwards -- and finally forms dq, the temporary
 * pairs, dx and every parameter gradient as products over all B*N rows at once.
 * Batches above 32 sequences run each step of the reverse loop as dense products over the batch (Sec. 6's regime).
 * The reverse loop and the attention terms are fp32 on CUDA cores; with bf16 storage the products over all rows run
 * on the tensor cores (operands rounded to bf16, fp32 accumulation).  recur_block > 1 returns RT_ERR_UNSUPPORTED.
 * The workspace needs rt_backward_workspace_bytes (about 40 fp32 arrays of B*N*d plus 4 of B*N*d_ff: 1.1 GB at B=4, N=2048, d=768; 48 GB at B=N=512, d=1024). */
typedef struct {
  float *w_q, *w_k, *w_v, *w_o, *w_up, *w_down;   /* shapes of rt_layer_weights */
  float *g_attn, *g_mlp, *g_kv, *g_q, *g_k;       /* [d_model] */
} rt_layer_grads;
size_t    rt_backward_workspace_bytes(const rt_config *cfg, int32_t B, int32_t N);
rt_status rt_layer_backward(const rt_config *cfg, const rt_layer_weights *w, const void *x, const void *z, const float *dz,
                            int32_t B, int32_t N, float *dx, const rt_layer_grads *grads,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Self-test of the bounded device-side wait (no counterpart in the paper): enqueues a two-CTA kernel
 * whose grid barrier expects an arrival that never comes.  The wait gives up after its limit (2 s),
 * the kernel returns normally, and rt_get_status(workspace) then reports RT_ERR_TIMEOUT; the CUDA
 * context stays usable.  `workspace` needs 256 bytes. */
rt_status rt_selftest_wait_expiry(void *workspace, void *cuda_stream);

/* Per-kernel-class timing for benchmarks.  While enabled (a process-wide switch, off by
 * default, and the one piece of global state in the library) every call brackets its launches
 * with CUDA events on the caller's stream: class 0 = pre-pass, 1 = leaf recurrence launches,
 * 2 = cross-block tiles, 3 = embedding / head.  rt_profile_read waits for the recorded events
 * (so call it after the work was enqueued), returns the summed milliseconds and the number of
 * bracketed launch groups per class since the last read, and forgets them.  on = 2 additionally makes
 * CTA 0 of the leaf kernels accumulate per-phase nanoseconds in the workspace's sync area (a diagnostic:
 * it slows the token step by a few per cent, because every phase waits for the slowest CTA).  The paper
 * has no counterpart; its latency protocol (Sec. 6, "The setup") times whole layers only. */
typedef struct { double ms[4]; uint64_t launches[4]; } rt_profile;
rt_status rt_profile_enable(int32_t on);
rt_status rt_profile_read(rt_profile *out);

/* The cross tiles of the tiled schedule for a length-N prefill with leaf size `leaf`
 * (Algorithm 1 applied to blocks of `leaf` positions), 0-based half-open:
 * tile i lets queries [q0,q1) attend to the pairs [k0,k1) right after position k1-1 is
 * revealed.  Writes up to `cap` entries of 4 int32 each to `out` (host) and returns the
 * number of tiles (call with cap = 0 to size the buffer).  Pure host function. */
int32_t rt_plan_tiles(int32_t N, int32_t leaf, int32_t *out, int32_t cap);

#ifdef __cplusplus
}
#endif
#endif /* RT_B200_H */
