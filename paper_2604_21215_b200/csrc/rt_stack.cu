// Embedding gather and the tied output head of the stack: x^0 = E[ids];
// logits = E . RMS_{g_final}(x^L) at one position per sequence.  The paper treats both as those
// of an ordinary Transformer (Sec. 6, "The setup") and leaves them out of its latency numbers.
#include "rt_kernels.h"

namespace rt {

template <typename T>
__global__ void embed_kernel(const T* emb, const int32_t* ids, long long n_tok, int d, int vocab, T* x) {
  const int per_row = d * (int)sizeof(T) / 16;          // 16-byte vectors per row
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_tok * per_row) return;
  const long long tok = i / per_row;
  const int v = (int)(i % per_row);
  int id = ids[tok];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);     // out-of-range ids are clamped, never dereferenced
  reinterpret_cast<uint4*>(x + tok * d)[v] = reinterpret_cast<const uint4*>(emb + (size_t)id * d)[v];
}

cudaError_t embed_launch(int dtype, const void* emb, const int32_t* ids, int B, int N, int d, int vocab, void* x,
                         cudaStream_t s) {
  const long long n_tok = (long long)B * N;
  const size_t es = dtype == RT_BF16 ? 2 : 4;
  const long long total = n_tok * (long long)(d * es / 16);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dtype == RT_BF16)
    embed_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((const __nv_bfloat16*)emb, ids, n_tok, d, vocab, (__nv_bfloat16*)x);
  else
    embed_kernel<float><<<blocks, 256, 0, s>>>((const float*)emb, ids, n_tok, d, vocab, (float*)x);
  return cudaGetLastError();
}

// One warp per vocabulary row: the row of E is read once and dotted with all B normalised
// hidden vectors (held in shared memory as fp32).
template <typename T>
__global__ void __launch_bounds__(256) head_kernel(const T* emb, const T* g_final, const T* hidden, long long h_bs,
                                                   int B, int d, int vocab, int norm_flags, float eps, float* logits) {
  extern __shared__ float hs[];                          // [B][d]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int b = warp; b < B; b += 8) {
    const T* hr = hidden + (size_t)b * h_bs;
    float ss = 0.f;
    for (int k = lane; k < d; k += 32) { const float v = to_f(hr[k]); ss += v * v; }
    ss = warp_sum(ss);
    const bool pre = (norm_flags & RT_NORM_PRE) != 0;
    const float rs = pre ? rsqrtf(ss / (float)d + eps) : 1.0f;
    for (int k = lane; k < d; k += 32) hs[b * d + k] = to_f(hr[k]) * rs * (pre ? gain_at(g_final, k) : 1.0f);
  }
  __syncthreads();
  for (int v = blockIdx.x * 8 + warp; v < vocab; v += gridDim.x * 8) {
    const T* er = emb + (size_t)v * d;
    for (int b0 = 0; b0 < B; b0 += 8) {
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int k = lane * 4; k < d; k += 128) {
        float f[4];
        reinterpret_cast<const Vec4<T>*>(er + k)->to_float(f);
#pragma unroll
        for (int bb = 0; bb < 8; ++bb) {
          if (b0 + bb < B) {
            const float4 a = *reinterpret_cast<const float4*>(hs + (b0 + bb) * d + k);
            acc[bb] += f[0] * a.x + f[1] * a.y + f[2] * a.z + f[3] * a.w;
          }
        }
      }
#pragma unroll
      for (int bb = 0; bb < 8; ++bb) {
        const float s = warp_sum(acc[bb]);
        if (lane == 0 && b0 + bb < B) logits[(size_t)(b0 + bb) * vocab + v] = s;
      }
    }
  }
}

cudaError_t head_launch(int dtype, const void* emb, const void* g_final, const void* hidden, long long h_bs, int B,
                        int d, int vocab, int norm_flags, float eps, float* logits, cudaStream_t s) {
  const size_t smem = sizeof(float) * (size_t)B * d;
  const int blocks = ceil_div(vocab, 8) < 1184 ? ceil_div(vocab, 8) : 1184;
  cudaError_t e;
  if (dtype == RT_BF16) {
    e = cudaFuncSetAttribute(head_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    head_kernel<__nv_bfloat16><<<blocks, 256, smem, s>>>((const __nv_bfloat16*)emb, (const __nv_bfloat16*)g_final,
                                                         (const __nv_bfloat16*)hidden, h_bs, B, d, vocab, norm_flags,
                                                         eps, logits);
  } else {
    e = cudaFuncSetAttribute(head_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    head_kernel<float><<<blocks, 256, smem, s>>>((const float*)emb, (const float*)g_final, (const float*)hidden, h_bs,
                                                 B, d, vocab, norm_flags, eps, logits);
  }
  return cudaGetLastError();
}

}  // namespace rt
