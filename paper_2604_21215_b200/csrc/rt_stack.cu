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

// bf16, B <= 16: the head as tensor-core mat-vecs.  The B normalised hidden rows sit in shared memory as TWO bf16 arrays
// (value = hi + lo, so the fp32 activations lose nothing that matters), the sequences are the 16 rows of an m16n8k16 MMA
// and 8 vocabulary rows its columns; a warp walks whole rows of E (each read once, 8 bytes per lane and k-step, 16 loads
// in flight) and writes 8 x B logits.  The kernel is bound by streaming E once.
__device__ __forceinline__ uint2 ldg_stream_v2(const void* p) {
  uint2 w;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w.x), "=r"(w.y) : "l"(p));
  return w;
}
__global__ void __launch_bounds__(256) head_mma_kernel(const __nv_bfloat16* emb, const __nv_bfloat16* g_final, const __nv_bfloat16* hidden,
                                                       long long h_bs, int B, int d, int vocab, int norm_flags, float eps, float* logits) {
  grid_dep_sync();                                           // chained to the last layer's kernel (programmatic dependent launch)
  extern __shared__ __align__(16) unsigned char hsm[];
  const int stride = d + 16;
  __nv_bfloat16* hi_s = reinterpret_cast<__nv_bfloat16*>(hsm);                 // [16][d + 16]
  __nv_bfloat16* lo_s = hi_s + (size_t)16 * stride;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool pre = (norm_flags & RT_NORM_PRE) != 0;
  for (int b = warp * 2; b < warp * 2 + 2; ++b) {
    __nv_bfloat16* hr_hi = hi_s + (size_t)b * stride;
    __nv_bfloat16* hr_lo = lo_s + (size_t)b * stride;
    if (b >= B) {
      for (int k = lane; k < d; k += 32) { hr_hi[k] = __float2bfloat16_rn(0.f); hr_lo[k] = __float2bfloat16_rn(0.f); }
      continue;
    }
    const __nv_bfloat16* hr = hidden + (size_t)b * h_bs;
    float ss = 0.f;
    for (int k = lane; k < d; k += 32) { const float v = __bfloat162float(hr[k]); ss += v * v; }
    ss = warp_sum(ss);
    const float rs = pre ? rsqrtf(ss / (float)d + eps) : 1.0f;
    for (int k = lane; k < d; k += 32) {
      const float v = __bfloat162float(hr[k]) * rs * (pre ? gain_at(g_final, k) : 1.0f);
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      hr_hi[k] = h;
      hr_lo[k] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
  __syncthreads();
  const int g = lane >> 2, c = lane & 3;
  const unsigned char* a_hi0 = reinterpret_cast<const unsigned char*>(hi_s + (size_t)g * stride + 4 * c);
  const unsigned char* a_hi1 = reinterpret_cast<const unsigned char*>(hi_s + (size_t)(g + 8) * stride + 4 * c);
  const unsigned char* a_lo0 = reinterpret_cast<const unsigned char*>(lo_s + (size_t)g * stride + 4 * c);
  const unsigned char* a_lo1 = reinterpret_cast<const unsigned char*>(lo_s + (size_t)(g + 8) * stride + 4 * c);
  const int n_ks = d / 16, n_groups = (vocab + 7) / 8;
  for (int grp = blockIdx.x * 8 + warp; grp < n_groups; grp += gridDim.x * 8) {
    const int v0 = grp * 8;
    const int vr = v0 + g < vocab ? v0 + g : vocab - 1;                        // rows beyond the vocabulary repeat the last one (not stored)
    const unsigned char* erow = reinterpret_cast<const unsigned char*>(emb + (size_t)vr * d + 4 * c);
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    for (int ks0 = 0; ks0 < n_ks; ks0 += 16) {
      uint2 bw[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) bw[i] = ldg_stream_v2(erow + (size_t)(ks0 + i < n_ks ? ks0 + i : ks0) * 32);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (ks0 + i < n_ks) {
          const size_t off = (size_t)(ks0 + i) * 32;
          const uint2 h0 = *reinterpret_cast<const uint2*>(a_hi0 + off), h1 = *reinterpret_cast<const uint2*>(a_hi1 + off);
          const uint2 l0 = *reinterpret_cast<const uint2*>(a_lo0 + off), l1 = *reinterpret_cast<const uint2*>(a_lo1 + off);
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(acc[0][0]), "+f"(acc[0][1]), "+f"(acc[0][2]), "+f"(acc[0][3])
                       : "r"(h0.x), "r"(h1.x), "r"(h0.y), "r"(h1.y), "r"(bw[i].x), "r"(bw[i].y));
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(acc[1][0]), "+f"(acc[1][1]), "+f"(acc[1][2]), "+f"(acc[1][3])
                       : "r"(l0.x), "r"(l1.x), "r"(l0.y), "r"(l1.y), "r"(bw[i].x), "r"(bw[i].y));
        }
      }
    }
    // acc[.][0], [1]: sequence g, vocabulary rows v0 + 2c, + 1; [2], [3]: sequence g + 8
    const int v = v0 + 2 * c;
    if (g < B) {
      if (v < vocab) logits[(size_t)g * vocab + v] = acc[0][0] + acc[1][0];
      if (v + 1 < vocab) logits[(size_t)g * vocab + v + 1] = acc[0][1] + acc[1][1];
    }
    if (g + 8 < B) {
      if (v < vocab) logits[(size_t)(g + 8) * vocab + v] = acc[0][2] + acc[1][2];
      if (v + 1 < vocab) logits[(size_t)(g + 8) * vocab + v + 1] = acc[0][3] + acc[1][3];
    }
  }
}

cudaError_t head_launch(int dtype, const void* emb, const void* g_final, const void* hidden, long long h_bs, int B,
                        int d, int vocab, int norm_flags, float eps, float* logits, cudaStream_t s) {
  const size_t smem = sizeof(float) * (size_t)B * d;
  const int blocks = ceil_div(vocab, 8) < 1184 ? ceil_div(vocab, 8) : 1184;
  cudaError_t e;
  if (dtype == RT_BF16 && B <= 16 && d % 16 == 0 && (size_t)2 * 16 * (d + 16) * 2 <= 200 * 1024) {
    const size_t sm2 = (size_t)2 * 16 * (d + 16) * 2;
    e = cudaFuncSetAttribute(head_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int groups = ceil_div(vocab, 8);
    const int nblk = ceil_div(groups, 8) < 2 * sms ? ceil_div(groups, 8) : 2 * sms;
    return launch_chained(head_mma_kernel, dim3(nblk), dim3(256), sm2, s, true, (const __nv_bfloat16*)emb, (const __nv_bfloat16*)g_final,
                          (const __nv_bfloat16*)hidden, h_bs, B, d, vocab, norm_flags, eps, logits);
  }
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
