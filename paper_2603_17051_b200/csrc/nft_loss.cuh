// Forward-process policy loss with selective KL, fused with its gradient: one pass over the four
// velocity tensors of the active window.  Pure bandwidth work (8 bytes read + 2 written per element):
// 16-byte vector loads, fp32 arithmetic, per-sample sums by warp shuffle + one atomic per block.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace astro {

constexpr int kNftThreads = 256;
constexpr int kNftVecsPerThread = 1;  // measured: one 16-byte vector per tensor and thread (many small blocks) is fastest

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// grid (blocks per sample, batch).  v_ref may be null (no KL term); grad may be null (loss only).
__global__ void __launch_bounds__(kNftThreads)
nft_loss_kernel(const uint4* __restrict__ v_theta, const uint4* __restrict__ v_old, const uint4* __restrict__ v_ref,
                const uint4* __restrict__ v_target, const float* __restrict__ r_tilde,
                const float* __restrict__ w_policy, const float* __restrict__ w_kl, const long long vecs_per_sample,
                const float beta, float* __restrict__ policy_out, float* __restrict__ kl_out,
                uint4* __restrict__ grad) {
  const int b = blockIdx.y;
  const float r = r_tilde[b];
  const float wp = w_policy ? w_policy[b] : 1.f, wk = (w_kl && v_ref) ? w_kl[b] : 0.f;
  const float gp = 2.f * beta * wp, gk = 2.f * wk;
  const long long base = static_cast<long long>(b) * vecs_per_sample;
  float sum_p = 0.f, sum_k = 0.f;
  const long long stride = static_cast<long long>(gridDim.x) * kNftThreads;
  for (long long v0 = static_cast<long long>(blockIdx.x) * kNftThreads + threadIdx.x; v0 < vecs_per_sample;
       v0 += stride * kNftVecsPerThread) {
    uint4 a[kNftVecsPerThread], o[kNftVecsPerThread], rf[kNftVecsPerThread], t[kNftVecsPerThread];
#pragma unroll
    for (int i = 0; i < kNftVecsPerThread; ++i) {
      const long long v = v0 + i * stride;
      if (v < vecs_per_sample) {
        a[i] = v_theta[base + v];
        o[i] = v_old[base + v];
        t[i] = v_target[base + v];
        if (v_ref) rf[i] = v_ref[base + v];
      }
    }
#pragma unroll
    for (int i = 0; i < kNftVecsPerThread; ++i) {
      const long long v = v0 + i * stride;
      if (v >= vecs_per_sample) continue;
      float fa[8], fo[8], ft[8], fr[8], g[8];
      bf16x8_to_f32(a[i], fa);
      bf16x8_to_f32(o[i], fo);
      bf16x8_to_f32(t[i], ft);
      if (v_ref) bf16x8_to_f32(rf[i], fr);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float d = fa[e] - fo[e];                 // v_theta - v_old
        const float ep = fmaf(beta, d, fo[e]) - ft[e];   // v+ - target
        const float en = fmaf(-beta, d, fo[e]) - ft[e];  // v- - target
        sum_p += r * ep * ep + (1.f - r) * en * en;
        float ge = gp * (r * ep - (1.f - r) * en);
        if (v_ref) {
          const float dk = fa[e] - fr[e];
          sum_k = fmaf(dk, dk, sum_k);
          ge = fmaf(gk, dk, ge);
        }
        g[e] = ge;
      }
      if (grad) {
        uint4 w;
        __nv_bfloat162* pw = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
        for (int e = 0; e < 4; ++e) pw[e] = __floats2bfloat162_rn(g[2 * e], g[2 * e + 1]);
        grad[base + v] = w;
      }
    }
  }
  __shared__ float red[2][kNftThreads / 32];
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    sum_p += __shfl_xor_sync(0xffffffffu, sum_p, s);
    sum_k += __shfl_xor_sync(0xffffffffu, sum_k, s);
  }
  if ((threadIdx.x & 31) == 0) {
    red[0][threadIdx.x >> 5] = sum_p;
    red[1][threadIdx.x >> 5] = sum_k;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    float p = threadIdx.x < kNftThreads / 32 ? red[0][threadIdx.x] : 0.f;
    float k = threadIdx.x < kNftThreads / 32 ? red[1][threadIdx.x] : 0.f;
#pragma unroll
    for (int s = 4; s > 0; s >>= 1) {
      p += __shfl_xor_sync(0xffffffffu, p, s);
      k += __shfl_xor_sync(0xffffffffu, k, s);
    }
    if (threadIdx.x == 0) {
      atomicAdd(policy_out + b, p);
      if (kl_out) atomicAdd(kl_out + b, k);
    }
  }
}

}  // namespace astro
